// ccoll_noalloc.cu — ccoll_compress_noalloc: ccoll_compress for callers that cannot hand the library any
// scratch memory.  The compress kernel needs a little global scratch beyond its input and output (one
// 8-byte size word per group of 4096 values, plus one per 32 groups, through which CTAs learn where their
// group starts in the stream).  The ordinary entry point takes it from the caller's registered workspace;
// this one takes it from a fixed array that lives in the library's own device image, so the call path
// contains no allocation of any kind.
#include "../../include/ccoll.h"
#include "ccoll_kernels.cuh"

#include <cmath>
#include <cstring>
#include <mutex>

namespace {

using namespace ccoll;

constexpr size_t kMaxGroups = CCOLL_NOALLOC_MAX_VALUES / kGroupValues;  // 16384
constexpr size_t kSizeWords = state_words((uint32_t)kMaxGroups);  // A[groups] + SA[groups / 32]

// The scratch itself.  Every GPU that loads the library holds these ~136 KB until the process exits.
// Zero at load time; later calls find the previous call's words in it (see the epoch below).
static __device__ __align__(256) unsigned long long g_size_words[kSizeWords];

struct PerDevice {
  uint64_t* words = nullptr;  // DEVICE address of g_size_words on that GPU (the symbol itself is only a host-side handle)
  uint32_t epoch = 0;
};
PerDevice g_dev[64];
std::mutex g_mu;

}  // namespace

extern "C" int ccoll_compress_noalloc(const float* in, size_t n, float abs_err_bound, uint32_t block_len, void* out,
                                      uint64_t* out_bytes, uint32_t* status, void* stream) {
  if (block_len != CCOLL_BLOCK_LEN) return CCOLL_ERR_UNSUPPORTED;
  if (n > CCOLL_NOALLOC_MAX_VALUES) return CCOLL_ERR_CAPACITY;  // the fixed scratch has no room for more groups
  uint32_t eb_bits;
  std::memcpy(&eb_bits, &abs_err_bound, 4);
  if (!std::isfinite(abs_err_bound) || !(abs_err_bound > 0.0f) || ((eb_bits >> 23) & 0xffu) == 0u)
    return CCOLL_ERR_INVALID_ARG;
  if (!out || !status || (!in && n) || (reinterpret_cast<uintptr_t>(in) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
      (reinterpret_cast<uintptr_t>(out_bytes) & 7u) || (reinterpret_cast<uintptr_t>(status) & 3u))
    return CCOLL_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CCOLL_ERR_CUDA;
  if (dev < 0 || dev >= 64) return CCOLL_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  std::lock_guard<std::mutex> lock(g_mu);
  PerDevice& d = g_dev[dev];
  if (!d.words) {
    // first call on this device: ask the runtime where the array lives on the GPU that is current now
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_size_words) != cudaSuccess || !p) return CCOLL_ERR_CUDA;
    d.words = static_cast<uint64_t*>(p);
  }
  // Size words carry the epoch of the launch that wrote them, so what the previous call left behind reads
  // as "not written yet" and nothing has to be cleared — except when the 32-bit epoch wraps around.
  if (++d.epoch == 0u) {
    if (cudaMemsetAsync(d.words, 0, kSizeWords * sizeof(uint64_t), s) != cudaSuccess) return CCOLL_ERR_CUDA;
    d.epoch = 1u;
  }

  EncodeBatch b;
  std::memset(&b, 0, sizeof(b));
  b.x = in;
  b.chunk_len = n ? n : 1;
  b.n = n;
  b.P = 1;
  b.sout = static_cast<uint8_t*>(out);
  b.out_cap = ccoll_compress_bound(n, block_len);
  b.out_bytes = out_bytes;
  b.moved_mult = 1;
  const size_t G = (((n + kL - 1) / kL) + kGroupBlocks - 1) / kGroupBlocks;
  b.tile_state = d.words;
  b.tiles_per_job = (uint32_t)G;
  b.state_stride = state_words((uint32_t)G);
  b.epoch = d.epoch;
  b.status = status;
  b.eb = abs_err_bound;
  b.eb_exp = (int)((eb_bits >> 23) & 0xffu);
  if (!launch_compress(b, (uint32_t)(G ? G : 1), 1, s)) return CCOLL_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? CCOLL_OK : CCOLL_ERR_CUDA;
}
