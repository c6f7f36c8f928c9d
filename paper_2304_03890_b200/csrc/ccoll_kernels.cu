// ccoll_kernels.cu — device code of libccoll (see ccoll_kernels.cuh for the work decomposition and
// include/ccoll.h for the stream layout and the block rules).  Compiled with --fmad=false: every fp32
// operation of the block rules rounds once, exactly as stated.
//
// Lane mapping (all kernels): thread tid of the CTA owns ROW tid of the group = 32 consecutive values
// (128 bytes); block = tid / 4, so four neighbouring lanes share a block and everything that must cross
// lanes (min/max, the predecessor code, byte offsets) is a two-step shuffle inside that quad of lanes.
// Per-value work runs serially inside a lane over eight 128-bit quads, so per-block quantities (mid-range,
// required bits, header) cost 4 lanes, not 32.
//
// Data movement: a group's fp32 values are a tile of 128 rows x 128 bytes in shared memory.  In the decoder
// and the fused round a complete group moves as one TMA tile (cp.async.bulk.tensor, 128-byte swizzle; loads
// complete on an mbarrier, stores are drained with wait_group.read), and the incoming payload as one bulk
// copy, so none of it passes through the load/store pipe; the encoder scatters coalesced 128-bit loads into
// rows padded to 144 bytes instead (cheaper for it than the swizzle's XOR per access).  (One 128-byte
// bulk-async copy per lane was measured first: a million such copies per 134 MB capped the kernel near
// 1.2 TB/s.)  Variable-length bytes are first appended to the lane's own row (aligned word stores), then
// copied once to their byte offset in a shared-memory image of the group's payload, which leaves as
// coalesced word stores at the offset that the two-level sum of the earlier groups' sizes yields.
#include "ccoll_kernels.cuh"

#include <cstdlib>
#include <cstring>
#include <utility>

#include <cuda.h>  // CUtensorMap and the enums of cuTensorMapEncodeTiled (types only; nothing links libcuda)

namespace ccoll {
#ifdef CCOLL_TIMELINE  // development aid: per-CTA phase timestamps (never compiled into the shipped library)
__device__ unsigned long long g_timeline[8192 * 16];
#define TL(slot)                                                                   \
  do {                                                                             \
    if (threadIdx.x == 0 && blockIdx.x < 8192 && blockIdx.y == 0 && blockIdx.z == 0) { \
      unsigned long long t_;                                                       \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                       \
      g_timeline[blockIdx.x * 16 + (slot)] = t_;                                    \
    }                                                                              \
  } while (0)
#else
#define TL(slot) do {} while (0)
#endif
namespace {
constexpr uint32_t kFull = 0xffffffffu;
constexpr int kSliceVals = 32;                      // values per lane
constexpr int kRowsBytes = kThreads * kSliceVals * 4;  // 16384: one 128-byte row per lane, no padding (swizzled)

// ---------------------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ float max_nan(float a, float b) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float min_nan(float a, float b) {
  float r;
  asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
// three-input forms (sm_100): fold two new values into a running extreme with one instruction
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float r;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float min3_nan(float a, float b, float c) {
  float r;
  asm("min.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// Byte permutation with a selector that is known to be well formed (every nibble 0..7): the intrinsic
// __byte_perm masks a run-time selector first, one more integer instruction per use.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ uint32_t mad_lo(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t opaque(uint32_t v) {  // hides a constant from the optimiser
  asm("" : "+r"(v));
  return v;
}
__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t* p) {
  uint64_t v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u64(uint64_t* p, uint64_t v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Programmatic dependent launch.  `grid_release` lets a grid launched behind this one (with the programmatic
// attribute) start filling SM slots as soon as every CTA of this grid has begun; `grid_acquire` holds such a grid
// until the grid before it has finished and its writes are visible.  Without the attribute both do nothing.
__device__ __forceinline__ void grid_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_acquire() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ uint64_t pack_state(uint32_t epoch, uint32_t flag, uint32_t value) {
  return ((uint64_t)epoch << 32) | ((uint64_t)flag << 30) | (uint64_t)(value & kValueMask);
}
__device__ __forceinline__ void raise(uint32_t* status, uint32_t code) { atomicMax(status, code); }
__device__ __forceinline__ uint32_t payload_base(uint32_t G) { return (kHeaderBytes + 8u * G + 4u + 15u) & ~15u; }

// unaligned reads from a word image in shared memory
__device__ __forceinline__ uint32_t img_u32(const uint32_t* img, uint32_t byte_off) {
  uint32_t w = byte_off >> 2;
  return __funnelshift_r(img[w], img[w + 1], 8u * (byte_off & 3u));
}
__device__ __forceinline__ uint32_t img_u8(const uint32_t* img, uint32_t byte_off) {
  return (img[byte_off >> 2] >> (8u * (byte_off & 3u))) & 0xffu;
}
// The outgoing image is zeroed once and its shared words are filled by atomic OR, so bytes of one word
// may come from any lane.
__device__ __forceinline__ void or_u8(uint32_t* img, uint32_t off, uint32_t byte) {
  atomicOr(&img[off >> 2], (byte & 0xffu) << (8u * (off & 3u)));
}
__device__ __forceinline__ void or_u32(uint32_t* img, uint32_t off, uint32_t v) {
  uint32_t z = 8u * (off & 3u), w = off >> 2;
  atomicOr(&img[w], v << z);
  if (z) atomicOr(&img[w + 1], v >> (32u - z));
}
__device__ __forceinline__ void or_u64(uint32_t* img, uint32_t off, uint32_t lo, uint32_t hi) {
  uint32_t z = 8u * (off & 3u), w = off >> 2;
  atomicOr(&img[w], lo << z);
  atomicOr(&img[w + 1], __funnelshift_l(lo, hi, z));
  if (z) atomicOr(&img[w + 2], hi >> (32u - z));
}

// ---------------------------------------------------------------------------------------------------
// geometry
// ---------------------------------------------------------------------------------------------------
struct JobGeom {
  uint32_t lo;      // first value of the job inside the rank buffer
  uint32_t len;     // values in the job
  uint32_t nb;      // blocks
  uint32_t G;       // groups
  uint32_t m_last;  // values in the job's last block (1..128; 0 if the job is empty)
};
// A rank buffer holds at most 2^29 values (the entry points check it), so value indices fit 32 bits.
__device__ __forceinline__ JobGeom job_geom(uint64_t n64, uint64_t C64, uint32_t y) {
  JobGeom j;
  const uint32_t n = (uint32_t)n64, C = (uint32_t)C64;
  const uint64_t lo64 = (uint64_t)y * C;
  j.lo = lo64 < n ? (uint32_t)lo64 : n;
  j.len = min(C, n - j.lo);
  j.nb = (j.len + kL - 1) / kL;
  j.G = (j.nb + kGroupBlocks - 1) / kGroupBlocks;
  j.m_last = j.len - (j.nb ? j.nb - 1 : 0) * kL;
  return j;
}
// What a thread owns in group g: its block's value count and its own valid values.
struct LaneGeom {
  uint32_t blk;    // block inside the group (tid / 4)
  uint32_t t;      // slice inside the block (tid % 4)
  uint32_t m_blk;  // values in the block (0 = the block does not exist)
  uint32_t nv;     // valid values in this lane's slice (0..32)
};
__device__ __forceinline__ LaneGeom lane_geom(const JobGeom& jg, uint32_t g) {
  LaneGeom lg;
  const uint32_t tid = threadIdx.x;
  lg.blk = tid >> 2;
  lg.t = tid & 3u;
  uint32_t gblk = g * kGroupBlocks + lg.blk;
  lg.m_blk = gblk < jg.nb ? (gblk == jg.nb - 1 ? jg.m_last : (uint32_t)kL) : 0u;
  int nv = (int)lg.m_blk - (int)(kSliceVals * lg.t);
  lg.nv = (uint32_t)(nv < 0 ? 0 : (nv > kSliceVals ? kSliceVals : nv));
  return lg;
}
// values of group g that exist (4096 except in the job's last group)
__device__ __forceinline__ uint32_t group_count(const JobGeom& jg, uint32_t g) {
  return min((uint32_t)kGroupValues, jg.len - g * (uint32_t)kGroupValues);
}

// ---------------------------------------------------------------------------------------------------
// shared memory
// ---------------------------------------------------------------------------------------------------
// Dynamic shared memory of a CTA: this control block, then one or two `rows` buffers of kRowsBytes (one
// padded 144-byte slice per thread: fp32 in, staged bytes, fp32 out).
struct Smem {
  alignas(128) uint32_t img[kImgWords];  // payload image of the incoming / outgoing group
  uint32_t blk_size[kGroupBlocks];       // record bytes, 0 = absent block
  uint32_t blk_R[kGroupBlocks];          // 0 = constant or absent block
  uint32_t prefix;                       // exclusive prefix of this group, in words
  uint32_t fail;
  alignas(8) uint64_t bar;               // mbarrier the TMA load of the rows completes on
  uint64_t bar_in;                       // mbarrier the bulk copy of the incoming payload completes on
};
constexpr int kCtlBytes = (sizeof(Smem) + 1023) / 1024 * 1024;  // the rows behind it need 1024-byte alignment
extern __shared__ __align__(1024) uint8_t dyn_smem[];
// decode kernel: image (aliased by the output rows) at offset 0, then its mbarrier
constexpr int kDecodeBarOffset = kRowsBytes > (int)sizeof(uint32_t) * kImgWords ? kRowsBytes : (int)sizeof(uint32_t) * kImgWords;

// The image is built with atomic ORs, so it must start as zeros.  Only its front (10 KB, more than most
// groups need) is cleared up front; a group whose payload turns out longer clears the rest once its size is
// known (zero_image_rest), at the price of one more barrier.
constexpr int kZeroFrontWords = 5 * 4 * kThreads;  // five 128-bit stores per thread
constexpr int kZeroSlackWords = 8;                 // words past the payload that placement may touch
__device__ __forceinline__ void zero_image(uint32_t* img) {  // a barrier must follow
  uint4* p = reinterpret_cast<uint4*>(img) + threadIdx.x;
#pragma unroll
  for (int r = 0; r < kZeroFrontWords / (4 * kThreads); ++r) p[r * kThreads] = make_uint4(0u, 0u, 0u, 0u);
}
__device__ __forceinline__ void zero_image_rest(uint32_t* img) {  // whole CTA; ends with a barrier
  for (int v = kZeroFrontWords / 4 + (int)threadIdx.x; v < kImgWords / 4; v += kThreads)
    reinterpret_cast<uint4*>(img)[v] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
}

// Ask L2 for the fp32 values of a group that a later CTA will load (one 128-byte line per thread).  Issued by
// the CTA that currently occupies the SM slot that later CTA will get, so its loads find the data in L2.
__device__ __forceinline__ void prefetch_group(const float* x, const JobGeom& jg, uint32_t g) {
  if (g >= jg.G) return;
  const uint32_t first = g * (uint32_t)kGroupValues + 32u * threadIdx.x;
  if (first < jg.len) asm volatile("prefetch.global.L2 [%0];" ::"l"(x + first));
}

// ---- rows: the group's values as a tile the TMA unit moves ---------------------------------------------
// A group of 4096 fp32 values is a tile of 128 rows x 128 bytes, row t = the 32 values of lane t.  The TMA unit
// moves such a tile between global and shared memory in one instruction, past the load/store pipe, and applies
// the 128-byte swizzle on the way: inside every 1024-byte span the 16-byte piece j of row r sits at piece
// j ^ (r & 7).  A lane that walks its own row piece by piece then meets no bank conflict although the rows
// are only 128 bytes apart (no padding).  Byte offset o < 128 of row t is at  128 t + (o ^ 16 (t & 7))  =
// (128 t + 16 (t & 7)) ^ o : one XOR per access.
struct Row {
  uint8_t* tile;  // the rows buffer (1024-byte aligned)
  uint32_t off;   // 128 t + 16 (t & 7)
  __device__ __forceinline__ float4 quad(uint32_t j) const {
    return *reinterpret_cast<const float4*>(tile + (off ^ (16u * j)));
  }
  __device__ __forceinline__ void set_quad(uint32_t j, const float4& v) const {
    *reinterpret_cast<float4*>(tile + (off ^ (16u * j))) = v;
  }
};
__device__ __forceinline__ Row row_of(uint8_t* rows, uint32_t t) { return Row{rows, 128u * t + 16u * (t & 7u)}; }
// The other way to keep a lane's walk over its row free of bank conflicts: rows 144 bytes apart, no swizzle, no
// XOR per access.  The TMA unit makes this layout too: a box 36 values wide over a tensor whose rows have 32
// lands as rows of 144 bytes (the four values past the row's end are out of bounds and arrive as zeros; a
// store does not write them).  The encoder and the fused round use it (their integer pipe is the busy one,
// and the spare words of a row let lanes stagger their staged output); the decoder's output tile is swizzled
// (16 KB instead of 18 KB: that is what lets 12 of its CTAs share an SM).  Same interface as Row.
constexpr int kPaddedRowBytes = 144;
constexpr int kPaddedRowsBytes = kThreads * kPaddedRowBytes;  // 18432
struct PaddedRow {
  static constexpr uint32_t kWords = 36u;
  // Staged words start `rot` words into the row: with rows 36 words apart, lanes l and l + 8 would otherwise
  // hit the same bank whenever they are at the same word; lane l's word w now sits in bank 4 l + l/8 + w.
  __device__ static __forceinline__ uint32_t rot(uint32_t t) { return (t >> 3) & 3u; }
  uint8_t* p;
  __device__ __forceinline__ float4 quad(uint32_t j) const { return *reinterpret_cast<const float4*>(p + 16u * j); }
  __device__ __forceinline__ void set_quad(uint32_t j, const float4& v) const { *reinterpret_cast<float4*>(p + 16u * j) = v; }
  __device__ __forceinline__ uint4 words4(uint32_t j) const { return *reinterpret_cast<const uint4*>(p + 16u * j); }
  __device__ __forceinline__ uint32_t word(uint32_t i) const { return *reinterpret_cast<const uint32_t*>(p + 4u * i); }
  __device__ __forceinline__ void set_word(uint32_t i, uint32_t v) const { *reinterpret_cast<uint32_t*>(p + 4u * i) = v; }
  __device__ __forceinline__ uint32_t* word_ptr(uint32_t i) const { return reinterpret_cast<uint32_t*>(p + 4u * i); }
};
template <class RowT>
__device__ __forceinline__ RowT make_row(uint8_t* rows, uint32_t t);
template <>
__device__ __forceinline__ PaddedRow make_row<PaddedRow>(uint8_t* rows, uint32_t t) {
  return PaddedRow{rows + kPaddedRowBytes * t};
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// generic-proxy writes to shared memory must be fenced before the TMA unit (async proxy) reads them
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// One thread: arm the barrier and ask the TMA unit for rows [row0, row0+128) of plane `plane` of the tensor.
__device__ __forceinline__ void tma_load_tile(const CUtensorMap* map, uint8_t* rows, uint64_t* bar, uint32_t row0,
                                              uint32_t plane, uint32_t tile_bytes) {
  const uint32_t b = smem_u32(bar);
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_proxy_async();
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(tile_bytes) : "memory");
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(rows)),
      "l"(map), "r"(0), "r"(row0), "r"(plane), "r"(b)
      : "memory");
}
// Every thread that will read the rows: wait for the tile (phase 0 of the barrier).  The wait is bounded;
// false = it gave up (the caller raises a time-out and does not touch the rows).
__device__ __forceinline__ bool tma_wait_tile(uint64_t* bar) {
  const uint32_t b = smem_u32(bar);
#pragma unroll 1
  for (uint32_t tries = 0; tries < (1u << 16); ++tries) {
    uint32_t done;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(done)
        : "r"(b)
        : "memory");
    if (done) return true;
  }
  return false;
}
// One thread: store the tile to rows [row0, row0+128) of plane `plane` of the tensor; the same thread then
// calls tma_store_wait() before shared memory is reused or the CTA exits (the tile has been read by then).
__device__ __forceinline__ void tma_store_tile(const CUtensorMap* map, const uint8_t* rows, uint32_t row0, uint32_t plane) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(map), "r"(0),
               "r"(row0), "r"(plane), "r"(smem_u32(rows))
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Padded rows: every warp reads 512 contiguous bytes per instruction (128-bit streaming loads) and scatters
// them; in round r thread tid moves the float4 number r*128 + tid of the group, piece (tid & 7) of row
// 16 r + tid / 8.  Zeros past the end of the data.  A __syncthreads must follow before the rows are read.
__device__ __forceinline__ void load_rows_padded(uint8_t* rows, const float* x, const JobGeom& jg, uint32_t g) {
  const uint32_t tid = threadIdx.x;
  const uint32_t cnt = group_count(jg, g);
  const float* src = x + (size_t)g * kGroupValues;
  float4* dst = reinterpret_cast<float4*>(rows + (tid >> 3) * kPaddedRowBytes + 16u * (tid & 7u));
  constexpr int kRoundStride = (kThreads / 8) * kPaddedRowBytes / 16;  // float4s between a thread's rounds
  if (cnt == (uint32_t)kGroupValues) {  // a complete group: no bounds to watch
    float4 t[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) t[r] = __ldcs(reinterpret_cast<const float4*>(src) + r * kThreads + tid);
#pragma unroll
    for (int r = 0; r < 8; ++r) dst[r * kRoundStride] = t[r];
    return;
  }
#pragma unroll 1
  for (int r = 0; r < 8; ++r) {
    const uint32_t f = (uint32_t)r * kThreads + tid;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (4u * f + 4u <= cnt) {
      v = __ldcs(reinterpret_cast<const float4*>(src) + f);
    } else {
      if (4u * f + 0u < cnt) v.x = __ldcs(src + 4u * f + 0u);
      if (4u * f + 1u < cnt) v.y = __ldcs(src + 4u * f + 1u);
      if (4u * f + 2u < cnt) v.z = __ldcs(src + 4u * f + 2u);
    }
    dst[r * kRoundStride] = v;
  }
}
// The same with every warp loading its own 32 rows (4 KB of the group): in round r lane l moves the float4
// number 256 w + 32 r + l, piece (l & 7) of row 32 w + 4 r + l / 8.  A warp then depends on its own loads only:
// a __syncwarp is enough before its lanes read their rows.
__device__ __forceinline__ void load_rows_padded_own(uint8_t* rows, const float* x, const JobGeom& jg, uint32_t g) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t cnt = group_count(jg, g);
  const float* src = x + (size_t)g * kGroupValues;
  const uint32_t f0 = 256u * warp + lane;  // the thread's float4 of round 0
  float4* dst = reinterpret_cast<float4*>(rows + (32u * warp + (lane >> 3)) * kPaddedRowBytes + 16u * (lane & 7u));
  constexpr int kRoundStride = 4 * kPaddedRowBytes / 16;  // float4s between a thread's rounds (four rows)
  if (cnt == (uint32_t)kGroupValues) {
    float4 t[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) t[r] = __ldcs(reinterpret_cast<const float4*>(src) + f0 + 32 * r);
#pragma unroll
    for (int r = 0; r < 8; ++r) dst[r * kRoundStride] = t[r];
    return;
  }
#pragma unroll 1
  for (int r = 0; r < 8; ++r) {
    const uint32_t f = f0 + 32u * (uint32_t)r;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (4u * f + 4u <= cnt) {
      v = __ldcs(reinterpret_cast<const float4*>(src) + f);
    } else {
      if (4u * f + 0u < cnt) v.x = __ldcs(src + 4u * f + 0u);
      if (4u * f + 1u < cnt) v.y = __ldcs(src + 4u * f + 1u);
      if (4u * f + 2u < cnt) v.z = __ldcs(src + 4u * f + 2u);
    }
    dst[r * kRoundStride] = v;
  }
}
// A swizzled tile without the TMA unit (a group that is not complete, or no tensor map): coalesced 128-bit
// streaming stores, bounds watched; thread tid moves the float4 number r*128 + tid in round r, which is piece
// (tid & 7) of row 16 r + tid / 8.  A __syncthreads must separate it from the writes of the rows.
__device__ __forceinline__ void store_rows(const uint8_t* rows, float* out, const JobGeom& jg, uint32_t g) {
  const uint32_t tid = threadIdx.x;
  const uint32_t cnt = group_count(jg, g);
  float* dst = out + (size_t)g * kGroupValues;
  const uint8_t* src = rows + 128u * (tid >> 3) + 16u * ((tid & 7u) ^ ((tid >> 3) & 7u));
#pragma unroll 1
  for (int r = 0; r < 8; ++r) {
    const uint32_t f = (uint32_t)r * kThreads + tid;
    const float4 t = *reinterpret_cast<const float4*>(src + 2048 * r);
    if (4u * f + 4u <= cnt) {
      __stcs(reinterpret_cast<float4*>(dst) + f, t);
    } else {
      if (4u * f + 0u < cnt) dst[4u * f + 0u] = t.x;
      if (4u * f + 1u < cnt) dst[4u * f + 1u] = t.y;
      if (4u * f + 2u < cnt) dst[4u * f + 2u] = t.z;
    }
  }
}
// The same from padded rows (fused round: the owner's sums of a group that is not complete).
__device__ __forceinline__ void store_rows_padded(const uint8_t* rows, float* out, const JobGeom& jg, uint32_t g) {
  const uint32_t tid = threadIdx.x;
  const uint32_t cnt = group_count(jg, g);
  float* dst = out + (size_t)g * kGroupValues;
  const float4* src = reinterpret_cast<const float4*>(rows + (tid >> 3) * kPaddedRowBytes + 16u * (tid & 7u));
  constexpr int kRoundStride = (kThreads / 8) * kPaddedRowBytes / 16;
#pragma unroll 1
  for (int r = 0; r < 8; ++r) {
    const uint32_t f = (uint32_t)r * kThreads + tid;
    const float4 t = src[r * kRoundStride];
    if (4u * f + 4u <= cnt) {
      __stcs(reinterpret_cast<float4*>(dst) + f, t);
    } else {
      if (4u * f + 0u < cnt) dst[4u * f + 0u] = t.x;
      if (4u * f + 1u < cnt) dst[4u * f + 1u] = t.y;
      if (4u * f + 2u < cnt) dst[4u * f + 2u] = t.z;
    }
  }
}
// Ragged rows: values past the end of the data are replaced by the block's first value, so that they
// cannot change min or max.  (The first value of block b is the first value of row 4b.)  Whole warp.
template <class RowT>
__device__ __forceinline__ void pad_ragged(uint8_t* rows, const LaneGeom& lg) {
  __syncwarp();
  if (lg.nv < (uint32_t)kSliceVals) {
    const uint32_t f = make_row<RowT>(rows, threadIdx.x & ~3u).word(0);
    const RowT row = make_row<RowT>(rows, threadIdx.x);
    for (uint32_t i = lg.nv; i < (uint32_t)kSliceVals; ++i) row.set_word(i, f);
  }
  __syncwarp();
}

// ---------------------------------------------------------------------------------------------------
// encode side
// ---------------------------------------------------------------------------------------------------
// Rules R1-R6 for the lane's block (the four lanes of a block compute the same plan).
struct Plan {
  uint32_t R;        // kept bits; 0 = constant (or absent) block, 32 = lossless
  uint32_t mu_bits;  // representative value
  float mu;
  uint32_t sh;       // 32 - R (0 when R is 0 or 32)
  uint32_t B;        // bytes per code
  bool lossless;
};

// Largest and smallest of the lane's 32 values (a NaN wins both), read from the lane's slice.  The loop is
// unrolled only twice: fully unrolled on register arrays the fused kernel outgrew the 32 KB instruction cache.
template <class RowT>
__device__ __forceinline__ void lane_minmax(const RowT& row, float& mx, float& mn) {
  float4 q = row.quad(0);
  mx = max3_nan(max_nan(q.x, q.y), q.z, q.w);
  mn = min3_nan(min_nan(q.x, q.y), q.z, q.w);
#pragma unroll 2
  for (int j = 1; j < 8; ++j) {
    q = row.quad(j);
    mx = max3_nan(max3_nan(mx, q.x, q.y), q.z, q.w);
    mn = min3_nan(min3_nan(mn, q.x, q.y), q.z, q.w);
  }
}
__device__ __forceinline__ Plan plan_block(float mx, float mn, const LaneGeom& lg, float eb, int eb_exp) {
  mx = max_nan(mx, __shfl_xor_sync(kFull, mx, 1));
  mn = min_nan(mn, __shfl_xor_sync(kFull, mn, 1));
  mx = max_nan(mx, __shfl_xor_sync(kFull, mx, 2));
  mn = min_nan(mn, __shfl_xor_sync(kFull, mn, 2));
  const float kInf = __uint_as_float(0x7f800000u);
  bool special = !(fabsf(mx) < kInf) || !(fabsf(mn) < kInf);  // NaN or Inf somewhere in the block
  float mu = __fadd_rn(__fmul_rn(0.5f, mn), __fmul_rn(0.5f, mx));
  uint32_t mub = __float_as_uint(mu);
  if ((mub << 1) == 0u) mub = 0u;  // a zero of either sign becomes +0
  mu = __uint_as_float(mub);
  float r = fmaxf(__fsub_rn(mx, mu), __fsub_rn(mu, mn));
  Plan p;
  if (lg.m_blk == 0u || (!special && r <= eb)) {
    p.R = 0u;
    p.mu_bits = mub;
    p.mu = mu;
    p.sh = 0u;
    p.B = 0u;
    p.lossless = false;
    return p;
  }
  int m_bits = (int)((__float_as_uint(r) >> 23) & 0xffu) - eb_exp + 1;
  p.lossless = special || m_bits >= 23;
  p.R = p.lossless ? 32u : (uint32_t)(9 + m_bits);
  p.mu_bits = p.lossless ? 0u : mub;
  p.mu = __uint_as_float(p.mu_bits);
  p.sh = 32u - p.R;
  p.B = (p.R + 7u) >> 3;
  return p;
}

__device__ __forceinline__ uint32_t code_of(float x, const Plan& p) {
  return __float_as_uint(p.lossless ? x : __fsub_rn(x, p.mu)) >> p.sh;
}

// Rules R7-R8 for the lane's 32 values.  The lane's byte string is built in a 64-bit big-endian accumulator
// (hi:lo; Tb = bits appended so far, the low Tb & 31 of them still waiting): a value's stored bytes are its low
// n = 8 * (stored bytes) bits, appended with two funnel shifts; whenever 32 bits are complete they leave as
// one word (byte-reversed, since the first byte of the stream is the most significant one).  n comes
// straight from the leading-zero count of (code xor predecessor); `fix` forces at least one stored byte when
// the field is 4 bytes wide (lead is capped at 3).  Values are read from the lane's row quad by quad and the
// staged words overwrite the row in place, which is safe because at most 16 bytes are staged per quad and
// quad j is read before anything is written at or behind its position.
// kGeneral = false: all 32 values valid, block not lossless (loop unrolled twice).  kGeneral = true: ragged
// rows (values past nv store nothing and have lead code 0) and lossless blocks, rolled.
template <bool kGeneral, class RowT>
__device__ __forceinline__ void emit_lane(const RowT& row, uint32_t R, uint32_t mu_bits, uint32_t nv, uint32_t prev,
                                          uint32_t& T_out, uint32_t& code_lo, uint32_t& code_hi) {
  const bool lossless = kGeneral && R == 32u;
  const uint32_t B = (R + 7u) >> 3, sh = 32u - R;
  const uint32_t fix = (B == 4u) ? 1u : 0u;
  const uint32_t unused = 4u - B;  // top bytes of the 32-bit code that the field does not have
  const float mu = __uint_as_float(mu_bits);
  uint32_t lo = 0u, hi = 0u, Tb = 0u;
  uint32_t clo = 0u, chi = 0u;
  const uint32_t rot = RowT::rot(threadIdx.x);  // staged word k goes to word rot + k of the row
  uint32_t* wp = row.word_ptr(rot);             // where the next completed word goes
  auto put = [&](uint32_t q, uint32_t sa) {
    const uint32_t n = 32u - sa;
    const uint32_t t = __funnelshift_lc(0u, q, sa);  // the stored bits, at the top of the word
    const uint32_t Tn = Tb + n;                      // the only loop-carried add: everything else hangs off it
    hi = __funnelshift_lc(lo, hi, n);
    lo = __funnelshift_lc(t, lo, n);
    if ((Tn ^ Tb) & 32u)  // a word boundary was crossed (n <= 32: at most one)
      *wp++ = __byte_perm(__funnelshift_r(lo, hi, Tn), 0u, 0x0123);
    Tb = Tn;
  };
  // the next quad is always read before the current one's words are stored: they may reach rot <= 3 words
  // into it
  float4 xn = row.quad(0);
#pragma unroll(kGeneral ? 1 : 2)
  for (int j = 0; j < 8; ++j) {
    const float4 x = xn;
    xn = row.quad(j < 7 ? j + 1 : 7);
    const uint32_t q0 = __float_as_uint(lossless ? x.x : __fsub_rn(x.x, mu)) >> sh,
                   q1 = __float_as_uint(lossless ? x.y : __fsub_rn(x.y, mu)) >> sh,
                   q2 = __float_as_uint(lossless ? x.z : __fsub_rn(x.z, mu)) >> sh,
                   q3 = __float_as_uint(lossless ? x.w : __fsub_rn(x.w, mu)) >> sh;
    uint32_t sa0 = (uint32_t)__clz((q0 ^ prev) | fix) & 0x38u, sa1 = (uint32_t)__clz((q1 ^ q0) | fix) & 0x38u,
             sa2 = (uint32_t)__clz((q2 ^ q1) | fix) & 0x38u, sa3 = (uint32_t)__clz((q3 ^ q2) | fix) & 0x38u;
    prev = q3;
    // lead code of a value = leading zero bytes of the xor, less the unused top bytes of the field; the
    // quad's four codes enter the 64-bit code string from the top, so that after eight quads quad 0 is lowest
    uint32_t cb;
    if (kGeneral) {
      uint32_t l0 = (sa0 >> 3) - unused, l1 = (sa1 >> 3) - unused, l2 = (sa2 >> 3) - unused, l3 = (sa3 >> 3) - unused;
      if (4u * j + 0u >= nv) sa0 = 32u, l0 = 0u;
      if (4u * j + 1u >= nv) sa1 = 32u, l1 = 0u;
      if (4u * j + 2u >= nv) sa2 = 32u, l2 = 0u;
      if (4u * j + 3u >= nv) sa3 = 32u, l3 = 0u;
      cb = (l0 | (l1 << 2) | (l2 << 4) | (l3 << 6)) << 24;
    } else {
      cb = ((sa0 + 4u * sa1 + 16u * sa2 + 64u * sa3) << 21) - unused * (85u << 24);
    }
    clo = __funnelshift_r(clo, chi, 8u);
    chi = (chi >> 8) | cb;
    put(q0, sa0);
    put(q1, sa1);
    put(q2, sa2);
    put(q3, sa3);
  }
  const uint32_t pend = Tb & 31u, w = Tb >> 5;
  // the last partial word, zero padded, and a zero word behind it for the realigning copy — as far as the row
  // reaches (a row that is full to its last byte has neither; copy_staged reads zeros past the row's end)
  if (rot + w < RowT::kWords) row.set_word(rot + w, pend ? __byte_perm(lo << (32u - pend), 0u, 0x0123) : 0u);
  if (rot + w + 1u < RowT::kWords) row.set_word(rot + w + 1u, 0u);
  T_out = Tb >> 3;
  code_lo = clo;
  code_hi = chi;
}
template <class RowT>
__device__ __noinline__ void emit_lane_general(RowT row, uint32_t R, uint32_t mu_bits, uint32_t nv, uint32_t prev,
                                               uint32_t& T_out, uint32_t& code_lo, uint32_t& code_hi) {
  emit_lane<true, RowT>(row, R, mu_bits, nv, prev, T_out, code_lo, code_hi);
}

// Copy the lane's T staged bytes (they start at word rot of its row) to byte offset dst of the image.  The
// first and last image word may be shared with a neighbour and are ORed in; the words between are plain
// stores.  The row is read in aligned 128-bit pieces from its start, as a string whose first rot words are
// to be skipped: row word g goes to image word (dst / 4) - rot + g.
template <class RowT>
__device__ __forceinline__ void copy_staged(uint32_t* img, const RowT& row, uint32_t dst, uint32_t T) {
  if (T == 0u) return;
  const uint32_t rot = RowT::rot(threadIdx.x);
  const uint32_t z = 8u * (dst & 3u);
  uint32_t* out = img + (dst >> 2);                // image word of staged word 0
  const uint32_t nw = ((dst & 3u) + T + 3u) >> 2;  // image words touched, <= 33
  atomicOr(&out[0], row.word(rot) << z);
  if (nw > 1u) {
    const uint32_t k = rot + nw - 1u;  // nothing is staged past the row's last word
    const uint32_t last = k < RowT::kWords ? row.word(k) : 0u;
    atomicOr(&out[nw - 1u], __funnelshift_l(row.word(k - 1u), last, z));
  }
  if (nw <= 2u) return;
  const uint32_t ni = nw - 2u;  // interior image words 1 .. nw-2 = row words rot+1 .. rot+nw-2
  uint32_t* outr = out - rot;   // image word of row word 0 (never dereferenced below row word rot + 1)
  uint32_t prevw = 0u;
  for (uint32_t c = 0; 4u * c <= rot + ni; ++c) {
    const uint4 cur = row.words4(c);
    const uint32_t w0 = __funnelshift_l(prevw, cur.x, z), w1 = __funnelshift_l(cur.x, cur.y, z),
                   w2 = __funnelshift_l(cur.y, cur.z, z), w3 = __funnelshift_l(cur.z, cur.w, z);
    prevw = cur.w;
    const uint32_t g = 4u * c - rot;  // staged word index of cur.x (wraps below zero for skipped words)
    if (g - 1u < ni) outr[4u * c] = w0;
    if (g < ni) outr[4u * c + 1u] = w1;
    if (g + 1u < ni) outr[4u * c + 2u] = w2;
    if (g + 2u < ni) outr[4u * c + 3u] = w3;
  }
}

// inclusive warp scan
__device__ __forceinline__ uint32_t warp_scan_u32(uint32_t v, uint32_t lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t t = __shfl_up_sync(kFull, v, d);
    if (lane >= (uint32_t)d) v += t;
  }
  return v;
}
// inclusive scan over the four lanes of a block; total = sum over the quad
__device__ __forceinline__ uint32_t quad_scan(uint32_t v, uint32_t t, uint32_t lane, uint32_t& total) {
  uint32_t a = __shfl_up_sync(kFull, v, 1);
  if (t >= 1u) v += a;
  a = __shfl_up_sync(kFull, v, 2);
  if (t >= 2u) v += a;
  total = __shfl_sync(kFull, v, lane | 3u);
  return v;
}

// Place of a group in its stream = sum of the sizes of all groups before it.  A chained look-back (wait
// for the predecessor's inclusive prefix) advances at most one window of tiles per L2 round trip, which
// caps a kernel of 8192 tiles at ~100 us whatever its work.  Instead sizes are summed on two levels and
// nothing ever waits on a prefix: A[t] = size of tile t; SA[s] = size of super-tile s (32 tiles), written
// by the super-tile's last tile from the A's it has to read anyway.  Tile g needs A[32s .. g-1] and
// SA[0 .. s-1]: independent loads spread over the CTA's threads, one round trip once the data is there.
// (A third level, sums of 1024 tiles, cuts the loads per tile from G/64 to about 36 and was measured slower.)
// Words carry the launch's epoch, so stale entries read as "not written yet"; every wait is bounded.
__device__ __forceinline__ uint32_t poll_size(const uint64_t* p, uint32_t epoch, uint32_t* status, bool& bad) {
  uint32_t spins = 0;
  while (true) {
    const uint64_t w = ld_relaxed_u64(p);
    if ((uint32_t)(w >> 32) == epoch) {
      if (((uint32_t)(w >> 30) & 3u) == kFlagPoison) bad = true;
      return (uint32_t)w & kValueMask;
    }
    if (++spins > kSpinLimit) {
      raise(status, kErrTimeout);
      bad = true;
      return 0u;
    }
    __nanosleep(32);
  }
}
// Both halves add to sm.prefix and raise sm.fail on a poisoned or timed-out entry; both words are read after
// the next barrier.  Called by every thread of the CTA after A[g] was published.
// Warp 0: the sizes of the earlier tiles of the own super-tile; the super-tile's last tile also publishes
// SA[s].  That tile calls this BEFORE it places its bytes in the image, every other tile after: the tiles of
// the next super-tile then find SA[s] one round trip after A[32s+31] instead of one placement and a round
// trip later.
struct SizeWords {
  uint64_t *A, *SA;
};
__device__ __forceinline__ SizeWords size_words(const EncodeBatch& b, uint32_t y) {
  SizeWords w;
  w.A = b.tile_state + (uint64_t)y * b.state_stride;
  w.SA = w.A + b.tiles_per_job;
  return w;
}
__device__ __forceinline__ void prefix_own_super_tile(Smem& sm, const SizeWords& w, uint32_t g, uint32_t G,
                                                      uint32_t words, uint32_t epoch, uint32_t* status) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  if (tid >= 32u) return;
  const uint32_t s = g >> 5, r = g & 31u;
  uint32_t sum = 0u;
  bool bad = false;
  if (lane < r) sum = poll_size(&w.A[32u * s + lane], epoch, status, bad);
  sum = __reduce_add_sync(kFull, sum);
  bad = __any_sync(kFull, bad);
  if (lane == 0) {
    if (r == 31u || g == G - 1u)
      st_relaxed_u64(&w.SA[s], pack_state(epoch, bad ? kFlagPoison : kFlagAggregate, sum + words));
    if (sum) atomicAdd(&sm.prefix, sum);
    if (bad) atomicOr(&sm.fail, 1u);
  }
}
// Warps 1-3: the earlier super-tiles.
__device__ __forceinline__ void prefix_earlier_super_tiles(Smem& sm, const SizeWords& w, uint32_t g, uint32_t epoch,
                                                           uint32_t* status) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  if (tid < 32u) return;
  const uint32_t s = g >> 5;
  uint32_t sum = 0u;
  bool bad = false;
  for (uint32_t t = tid - 32u; t < s; t += kThreads - 32u) sum += poll_size(&w.SA[t], epoch, status, bad);
  sum = __reduce_add_sync(kFull, sum);
  bad = __any_sync(kFull, bad);
  if (lane == 0) {
    if (sum) atomicAdd(&sm.prefix, sum);
    if (bad) atomicOr(&sm.fail, 1u);
  }
}

// Encode the group whose values wait in the lanes' slices (ragged slices already padded; mx, mn = largest and
// smallest value of the lane's slice): build the payload image, find its place in the stream and copy it
// out.  The image must have been zeroed (that is made visible by the barrier inside) before the call.
template <class RowT>
__device__ __forceinline__ void encode_group(Smem& sm, uint8_t* rows, const LaneGeom& lg, const EncodeBatch& b,
                                             const JobGeom& jg, uint32_t g, uint32_t y, uint8_t* sout, float mx,
                                             float mn, bool tail) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const RowT row = make_row<RowT>(rows, tid);
  Plan p = plan_block(mx, mn, lg, b.eb, b.eb_exp);
  // code of the value just before this lane's first one (0 at the start of a block)
  uint32_t prev = __shfl_up_sync(kFull, code_of(__uint_as_float(row.word(kSliceVals - 1)), p), 1);
  if (lg.t == 0u) prev = 0u;
  uint32_t T = 0u, code_lo = 0u, code_hi = 0u;
  if (p.R != 0u) {
    if (tail || p.lossless)
      emit_lane_general(row, p.R, p.mu_bits, lg.nv, prev, T, code_lo, code_hi);
    else
      emit_lane<false, RowT>(row, p.R, p.mu_bits, (uint32_t)kSliceVals, prev, T, code_lo, code_hi);
  }
  uint32_t total;
  const uint32_t excl = quad_scan(T, lg.t, lane, total) - T;
  const uint32_t cbytes = (lg.m_blk + 3u) >> 2;  // lead-code bytes of the block
  if (lg.t == 0u) {
    sm.blk_size[lg.blk] = lg.m_blk == 0u ? 0u : (p.R ? 5u + cbytes + total : 4u);
    sm.blk_R[lg.blk] = p.R;
  }
  __syncthreads();  // sizes visible; also: image zero-fill and all staging done
  TL(4);

  // every warp derives the offsets of all 32 records (cheap, and saves a barrier)
  const uint32_t sz_l = sm.blk_size[lane];
  const uint32_t R_l = sm.blk_R[lane];
  const uint32_t bitmap = __ballot_sync(kFull, R_l != 0u);
  const uint32_t k = (uint32_t)__popc(bitmap);
  const uint32_t incl_sz = warp_scan_u32(sz_l, lane);
  const uint32_t off_l = 2u * k + incl_sz - sz_l;
  const uint32_t raw = 2u * k + __shfl_sync(kFull, incl_sz, 31);
  const uint32_t words = (raw + 3u) >> 2;
  const uint32_t boff = __shfl_sync(kFull, off_l, lg.blk);
  if (words + (uint32_t)kZeroSlackWords > (uint32_t)kZeroFrontWords) zero_image_rest(sm.img);  // rare, uniform

  const SizeWords sw = size_words(b, y);
  if (warp == 0) {
    if (lane == 0) st_relaxed_u64(&sw.A[g], pack_state(b.epoch, kFlagAggregate, words));
    if (R_l != 0u) {
      uint32_t rank = (uint32_t)__popc(bitmap & ((1u << lane) - 1u));
      atomicOr(&sm.img[rank >> 1], sz_l << (16u * (rank & 1u)));
    }
  }
  const bool closes = (g & 31u) == 31u || g == jg.G - 1u;  // this tile completes its super-tile
  if (closes) prefix_own_super_tile(sm, sw, g, jg.G, words, b.epoch, b.status);
  if (lg.m_blk != 0u) {
    if (lg.t == 0u) {
      or_u32(sm.img, boff, p.mu_bits);
      if (p.R) or_u8(sm.img, boff + 4u, p.R);
    }
    if (p.R) {
      if (8u * lg.t < cbytes) or_u64(sm.img, boff + 5u + 8u * lg.t, code_lo, code_hi);
      copy_staged(sm.img, row, boff + 5u + cbytes + excl, T);
    }
  }

  // place of the group in the stream
  TL(5);
  if (!closes) prefix_own_super_tile(sm, sw, g, jg.G, words, b.epoch, b.status);
  prefix_earlier_super_tiles(sm, sw, g, b.epoch, b.status);
  TL(11);
  __syncthreads();
  TL(6);
  const uint32_t prefix = sm.prefix;
  if (sm.fail) return;
  const uint32_t base = payload_base(jg.G);
  const uint64_t end = (uint64_t)base + 4ull * ((uint64_t)prefix + words);
  uint32_t* out32 = reinterpret_cast<uint32_t*>(sout);
  if (end > b.out_cap) {
    if (tid == 0) raise(b.status, kErrCapacity);
    return;
  }
  {
    // coalesced copy-out: consecutive lanes move consecutive words (conflict-free shared reads, full
    // 128-byte lines per warp store)
    uint32_t* dst = out32 + (base >> 2) + prefix;
    TL(8);
    for (uint32_t j = tid; j < words; j += kThreads) __stcs(dst + j, sm.img[j]);
    TL(9);
  }
  if (tid == 0) {
    out32[8 + g] = prefix;             // dir[g]
    out32[8 + jg.G + 1 + g] = bitmap;  // bitmap[g]
  }
  TL(10);
  if (g == 0 && tid >= 32 && tid < 32 + 4) {
    // static part of the header and the zero pad between the bitmap and the payload
    uint32_t t = tid - 32;
    if (t == 0) {
      out32[0] = kMagic;
      out32[1] = 0u;
      out32[2] = jg.len;
      out32[3] = 0u;
      out32[4] = (uint32_t)kL;
      out32[5] = __float_as_uint(b.eb);
    }
    for (uint32_t w = 8 + 2 * jg.G + 1 + t; w < (base >> 2); w += 4) out32[w] = 0u;
  }
  if (g == jg.G - 1 && tid == 64) {
    out32[8 + jg.G] = prefix + words;  // dir[G]
    out32[6] = (uint32_t)end;
    out32[7] = (uint32_t)(end >> 32);
    if (b.out_bytes) b.out_bytes[y] = end;
    if (b.moved) atomicAdd(reinterpret_cast<unsigned long long*>(b.moved), (unsigned long long)b.moved_mult * end);
  }
}

// An empty job still yields a valid 48-byte stream.
__device__ __forceinline__ void write_empty_stream(const EncodeBatch& b, uint32_t y, uint8_t* sout) {
  if (threadIdx.x != 0) return;
  if (b.out_cap < 48u) {
    raise(b.status, kErrCapacity);
    return;
  }
  uint32_t* out32 = reinterpret_cast<uint32_t*>(sout);
  out32[0] = kMagic;
  out32[1] = 0u;
  out32[2] = 0u;
  out32[3] = 0u;
  out32[4] = (uint32_t)kL;
  out32[5] = __float_as_uint(b.eb);
  out32[6] = 48u;
  out32[7] = 0u;
  out32[8] = 0u;  // dir[0]
  out32[9] = out32[10] = out32[11] = 0u;
  if (b.out_bytes) b.out_bytes[y] = 48u;
  if (b.moved) atomicAdd(reinterpret_cast<unsigned long long*>(b.moved), (unsigned long long)b.moved_mult * 48ull);
}

// ---------------------------------------------------------------------------------------------------
// decode side
// ---------------------------------------------------------------------------------------------------
struct StreamView {
  const uint32_t* words;  // the stream as 32-bit words
  uint32_t G, base;       // groups, payload_base
  uint32_t a, gw, map;    // first payload word of the group, its length in words, its bitmap
  uint32_t pw;            // payload words of the whole stream
};

// Validate the header and the directory entries of group g.  Every thread of the CTA reads the same words
// and reaches the same verdict.
__device__ __forceinline__ bool open_group(const uint8_t* sin, uint64_t in_bytes, const JobGeom& jg, uint32_t g,
                                           StreamView& sv) {
  sv.words = reinterpret_cast<const uint32_t*>(sin);
  sv.G = jg.G;
  sv.base = payload_base(jg.G);
  if (in_bytes < sv.base) return false;
  const uint32_t* w = sv.words;
  uint64_t n = (uint64_t)__ldg(w + 2) | ((uint64_t)__ldg(w + 3) << 32);
  uint64_t total = (uint64_t)__ldg(w + 6) | ((uint64_t)__ldg(w + 7) << 32);
  if (__ldg(w) != kMagic || __ldg(w + 1) != 0u || n != jg.len || __ldg(w + 4) != (uint32_t)kL) return false;
  if (total > in_bytes || total < sv.base || ((total - sv.base) & 3u)) return false;
  uint64_t pw = (total - sv.base) >> 2;  // payload words
  uint32_t a = __ldg(w + 8 + g), e = __ldg(w + 8 + g + 1);
  sv.map = __ldg(w + 8 + jg.G + 1 + g);
  if (a > e || (uint64_t)e > pw || (e - a) * 4u > (uint32_t)kMaxGroupBytes) return false;
  if (g == jg.G - 1 && (uint64_t)e != pw) return false;
  uint32_t nblk = min((uint32_t)kGroupBlocks, jg.nb - g * kGroupBlocks);
  if (nblk < 32u && (sv.map >> nblk) != 0u) return false;
  sv.a = a;
  sv.gw = e - a;
  sv.pw = (uint32_t)pw;
  return true;
}

// sum of the sixteen 2-bit fields of a word
__device__ __forceinline__ uint32_t sum_fields(uint32_t w) {
  return (uint32_t)__popc(w & 0x55555555u) + 2u * (uint32_t)__popc(w & 0xaaaaaaaau);
}

// One byte position of a lane's summary.  The lane's 32 lead codes sit in two words (values 0-15 in lo,
// 16-31 in hi).  Values with lead <= KB store byte KB of the field (counted from its most significant
// byte); the last such value is found with one leading-zero count, the stored bytes before it with two
// population counts, and its byte is fetched from the image.
struct SummaryIn {
  uint32_t lo, hi, lo1, hi1;  // the codes, and the codes shifted right by one
  uint32_t vlo, vhi;          // marker bit (even positions) of every valid value
  uint32_t lead_lo;           // sum of the leads of values 0-15
  uint32_t B, pos0;
};
template <int KB>
__device__ __forceinline__ void summary_byte(const uint32_t* img, const SummaryIn& si, uint32_t& sval, uint32_t& smask) {
  uint32_t ph, pl;  // markers of the values that store byte KB
  if (KB == 0) {
    ph = ~(si.hi | si.hi1) & si.vhi;
    pl = ~(si.lo | si.lo1) & si.vlo;
  } else if (KB == 1) {
    ph = ~si.hi1 & si.vhi;
    pl = ~si.lo1 & si.vlo;
  } else if (KB == 2) {
    ph = ~(si.hi & si.hi1) & si.vhi;
    pl = ~(si.lo & si.lo1) & si.vlo;
  } else {
    ph = si.vhi;
    pl = si.vlo;
  }
  if ((ph | pl) == 0u) return;
  const bool up = ph != 0u;
  const uint32_t pm = up ? ph : pl, w = up ? si.hi : si.lo;
  const uint32_t i2 = 31u - (uint32_t)__clz((int)pm);  // bit position of the value's code = 2 * (its index in the half)
  const uint32_t below = w & ((1u << i2) - 1u);        // codes of the values before it in this half
  const uint32_t lead_sum = (up ? si.lead_lo : 0u) + sum_fields(below);
  const uint32_t lead_i = (w >> i2) & 3u;
  const uint32_t i = (i2 >> 1) + (up ? 16u : 0u);
  const uint32_t byte = img_u8(img, si.pos0 + (si.B * i - lead_sum) + ((uint32_t)KB - lead_i));
  const uint32_t shift = 8u * (si.B - 1u - (uint32_t)KB);
  sval |= byte << shift;
  smask |= 0xffu << shift;
}

// One quad of the general decode path: any field width, lossless blocks, ragged slices (nvq = valid values
// of the quad).  Out of line on purpose (rare, and it keeps the kernels' hot code small).
struct DecodeCursor {
  uint32_t pos;   // image offset of the next stored byte
  uint32_t prev;  // code of the previous value
};
__device__ __noinline__ float4 decode_quad_generic(const uint32_t* img, DecodeCursor& cur, uint32_t cb, uint32_t R,
                                                   float mu, uint32_t nvq) {
  const uint32_t B = (R + 7u) >> 3, sh = 32u - R;
  uint32_t nb0 = B - (cb & 3u), nb1 = B - ((cb >> 2) & 3u), nb2 = B - ((cb >> 4) & 3u), nb3 = B - ((cb >> 6) & 3u);
  if (nvq < 1u) nb0 = 0u;
  if (nvq < 2u) nb1 = 0u;
  if (nvq < 3u) nb2 = 0u;
  if (nvq < 4u) nb3 = 0u;
  // the quad's stored bytes as a little-endian 16-byte string
  const uint32_t wi = cur.pos >> 2, z = 8u * (cur.pos & 3u);
  const uint32_t A0 = img[wi], A1 = img[wi + 1], A2 = img[wi + 2], A3 = img[wi + 3], A4 = img[wi + 4];
  const uint32_t S0 = __funnelshift_r(A0, A1, z), S1 = __funnelshift_r(A1, A2, z), S2 = __funnelshift_r(A2, A3, z),
                 S3 = __funnelshift_r(A3, A4, z);
  cur.pos += nb0 + nb1 + nb2 + nb3;
  // peel the four values off the front of the string
  const uint32_t c0 = 8u * nb0, c1 = 8u * nb1, c2 = 8u * nb2, c3 = 8u * nb3;
  const uint32_t U0 = __funnelshift_rc(S0, S1, c0), U1 = __funnelshift_rc(S1, S2, c0), U2 = __funnelshift_rc(S2, S3, c0);
  const uint32_t X0 = __funnelshift_rc(U0, U1, c1), X1 = __funnelshift_rc(U1, U2, c1);
  const uint32_t r3 = __funnelshift_rc(X0, X1, c2);
  // stored bytes as a right-aligned big-endian value; the bytes not stored come from the predecessor
  const uint32_t v0 = __funnelshift_rc(__byte_perm(S0, 0u, 0x0123), 0u, 32u - c0);
  const uint32_t v1 = __funnelshift_rc(__byte_perm(U0, 0u, 0x0123), 0u, 32u - c1);
  const uint32_t v2 = __funnelshift_rc(__byte_perm(X0, 0u, 0x0123), 0u, 32u - c2);
  const uint32_t v3 = __funnelshift_rc(__byte_perm(r3, 0u, 0x0123), 0u, 32u - c3);
  const uint32_t q0 = v0 | (cur.prev & ~__funnelshift_rc(kFull, 0u, 32u - c0));
  const uint32_t q1 = v1 | (q0 & ~__funnelshift_rc(kFull, 0u, 32u - c1));
  const uint32_t q2 = v2 | (q1 & ~__funnelshift_rc(kFull, 0u, 32u - c2));
  const uint32_t q3 = v3 | (q2 & ~__funnelshift_rc(kFull, 0u, 32u - c3));
  cur.prev = q3;
  if (R == 32u) return make_float4(__uint_as_float(q0), __uint_as_float(q1), __uint_as_float(q2), __uint_as_float(q3));
  return make_float4(__fadd_rn(__uint_as_float(q0 << sh), mu), __fadd_rn(__uint_as_float(q1 << sh), mu),
                     __fadd_rn(__uint_as_float(q2 << sh), mu), __fadd_rn(__uint_as_float(q3 << sh), mu));
}

// One reduction of the collective-computation framework (Sec. III-B): a = decoded value, b = local value.
// Sum: one rounded add (a NaN result is the GPU's canonical 0x7FFFFFFF).  Max / Min: a pure selection, a if
// it beats b or b is a NaN, else b.  kDivide (the owner's round of an Average, a kernel of its own so that the
// division costs the other rounds nothing): the sum, then one correctly rounded division by the number of
// ranks; a NaN quotient is made the same canonical NaN.
template <bool kDivide>
__device__ __forceinline__ float reduce_op(float a, float b, int op, float divisor) {
  if (kDivide) {
    const float q = __fdiv_rn(__fadd_rn(a, b), divisor);
    return q != q ? __uint_as_float(0x7fffffffu) : q;
  }
  if (op == 0) return __fadd_rn(a, b);
  if (op == 1) return (a > b || b != b) ? a : b;
  return (a < b || b != b) ? a : b;
}

// Decode the lane's 32 values of group g into v[].  Returns false (for the whole CTA) on a corrupt group.
// The group's payload must already be staged in sm.img (and visible).  nblk = blocks in the group.
// kToSlice = false: the values are returned in v[] (fully unrolled loops).  kToSlice = true (fused reduce):
// each decoded quad is REDUCED (op) with the quad of local values waiting in the lane's slice and the result is written
// back there, and mx / mn receive the largest / smallest result of the lane (meaningless for a ragged slice);
// the loops are then unrolled only twice, which keeps the fused kernel inside the instruction cache.
template <bool kToSlice, bool kDivide = false, class RowT = Row>
__device__ __forceinline__ bool decode_group(Smem& sm, const StreamView& sv, const LaneGeom& lg, uint32_t nblk,
                                             float4 (&v)[8], const RowT& row, int op, float divisor, float& mx,
                                             float& mn) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const uint32_t* img = sm.img + (sv.a & 3u);  // see stage_payload
  const bool tail = __any_sync(kFull, lg.nv != (uint32_t)kSliceVals);

  // offsets of the 32 records: lane b looks at block b
  bool bad = false;
  const uint32_t map = sv.map;
  const uint32_t k = (uint32_t)__popc(map);
  uint32_t sz_l = 0u;
  if (lane < nblk) {
    if ((map >> lane) & 1u) {
      uint32_t rank = (uint32_t)__popc(map & ((1u << lane) - 1u));
      sz_l = (rank < 2u * sv.gw) ? reinterpret_cast<const uint16_t*>(img)[rank] : 0u;
    } else {
      sz_l = 4u;
    }
  }
  const uint32_t incl_sz = warp_scan_u32(sz_l, lane);
  const uint32_t off_l = 2u * k + incl_sz - sz_l;
  const uint32_t raw = 2u * k + __shfl_sync(kFull, incl_sz, 31);
  if (((raw + 3u) >> 2) != sv.gw) bad = true;  // the same verdict in every thread
  const uint32_t boff = __shfl_sync(kFull, off_l, lg.blk);
  const uint32_t size_blk = __shfl_sync(kFull, sz_l, lg.blk);
  const bool nonconst = lg.m_blk != 0u && ((map >> lg.blk) & 1u);

  // header, lead codes and stored-byte count of the lane
  uint32_t R = 0u, B = 0u, code_lo = 0u, code_hi = 0u, T = 0u, lead_lo = 0u;
  const uint32_t cbytes = (lg.m_blk + 3u) >> 2;
  if (!bad && nonconst) {
    R = img_u8(img, boff + 4u);
    if (!(R >= 10u && R <= 32u)) bad = true;
    B = (R + 7u) >> 3;
    if (8u * lg.t < cbytes) {
      uint32_t o = boff + 5u + 8u * lg.t;
      uint32_t w = o >> 2, z = 8u * (o & 3u);
      uint32_t a0 = img[w], a1 = img[w + 1], a2 = img[w + 2];
      code_lo = __funnelshift_r(a0, a1, z);
      code_hi = __funnelshift_r(a1, a2, z);
      if (tail) {
        // only cbytes code bytes exist; codes of values past the end must be zero
        uint32_t vb = cbytes - 8u * lg.t;  // valid code bytes of this lane (>= 1)
        if (vb < 8u) {
          if (vb <= 4u) {
            code_hi = 0u;
            if (vb < 4u) code_lo &= (1u << (8u * vb)) - 1u;
          } else {
            code_hi &= (1u << (8u * (vb - 4u))) - 1u;
          }
        }
        if (lg.nv < (uint32_t)kSliceVals) {
          uint64_t c = ((uint64_t)code_hi << 32) | code_lo;
          if (c >> (2u * lg.nv)) bad = true;
        }
      }
    }
    if (B == 2u && ((code_lo & (code_lo >> 1) & 0x55555555u) | (code_hi & (code_hi >> 1) & 0x55555555u)))
      bad = true;  // lead 3 cannot occur in a 2-byte field
    lead_lo = sum_fields(code_lo);
    T = B * lg.nv - lead_lo - sum_fields(code_hi);
    if (bad) T = 0u;
  }
  uint32_t total;
  const uint32_t excl = quad_scan(T, lg.t, lane, total) - T;
  if (nonconst && !bad && size_blk != 5u + cbytes + total) bad = true;
  TL(12);
  if (__syncthreads_or(bad ? 1 : 0)) return false;
  TL(13);

  // Summary of the lane's values for the predecessor chain: for each byte of the code field, the byte the
  // LAST value of the lane that stores it holds (found from the lead codes alone, then fetched).
  const uint32_t pos0 = boff + 5u + cbytes + excl;  // image offset of the lane's first stored byte
  uint32_t sval = 0u, smask = 0u;
  if (nonconst && lg.nv != 0u) {
    SummaryIn si;
    si.lo = code_lo;
    si.hi = code_hi;
    si.lo1 = code_lo >> 1;
    si.hi1 = code_hi >> 1;
    si.vlo = 0x55555555u;  // one marker bit per valid value
    si.vhi = 0x55555555u;
    if (tail) {
      si.vlo = lg.nv < 16u ? ((1u << (2u * lg.nv)) - 1u) & 0x55555555u : 0x55555555u;
      si.vhi = lg.nv <= 16u ? 0u : (lg.nv < 32u ? ((1u << (2u * (lg.nv - 16u))) - 1u) & 0x55555555u : 0x55555555u);
    }
    si.lead_lo = lead_lo;
    si.B = B;
    si.pos0 = pos0;
    summary_byte<0>(img, si, sval, smask);
    if (B > 1u) summary_byte<1>(img, si, sval, smask);
    if (B > 2u) summary_byte<2>(img, si, sval, smask);
    if (B > 3u) summary_byte<3>(img, si, sval, smask);
  }
  // carry the summaries across the quad: what a lane does not store itself comes from its left
  {
    uint32_t tv = __shfl_up_sync(kFull, sval, 1), tm = __shfl_up_sync(kFull, smask, 1);
    if (lg.t >= 1u) {
      sval |= tv & ~smask;
      smask |= tm;
    }
    tv = __shfl_up_sync(kFull, sval, 2);
    tm = __shfl_up_sync(kFull, smask, 2);
    if (lg.t >= 2u) {
      sval |= tv & ~smask;
      smask |= tm;
    }
  }
  uint32_t prev = __shfl_up_sync(kFull, sval, 1);
  if (lg.t == 0u) prev = 0u;
  TL(14);

  // the lane's 32 values
  const float mu = (lg.m_blk != 0u) ? __uint_as_float(img_u32(img, boff)) : 0.0f;
  constexpr int kUnroll = kToSlice ? 2 : 8;
  auto put = [&](int j, const float4& r) {
    if (kToSlice) {
      const float4 a = row.quad(j);
      const float4 o = make_float4(reduce_op<kDivide>(r.x, a.x, op, divisor), reduce_op<kDivide>(r.y, a.y, op, divisor),
                                   reduce_op<kDivide>(r.z, a.z, op, divisor), reduce_op<kDivide>(r.w, a.w, op, divisor));
      row.set_quad(j, o);
      mx = max3_nan(max3_nan(mx, o.x, o.y), o.z, o.w);  // the encoder's min/max, while the values are at hand
      mn = min3_nan(min3_nan(mn, o.x, o.y), o.z, o.w);
    } else {
      v[j] = r;
    }
  };
  if (!nonconst) {
#pragma unroll kUnroll
    for (int j = 0; j < 8; ++j) put(j, make_float4(mu, mu, mu, mu));
    return true;
  }
  const uint64_t codes = ((uint64_t)code_hi << 32) | code_lo;
  const uint32_t sh = 32u - R;
  uint32_t pos = pos0;
  if (!tail && R <= 24u) {
    // Fast path: complete slice, field of at most 3 bytes.  A value is assembled by ONE byte permutation of
    // (predecessor, next four stream bytes): it takes the top `lead` bytes of the field from the predecessor
    // and the stored bytes, most significant first, from the stream.  The permutation depends only on the
    // number of stored bytes nb (0..3) and is itself picked, by a byte permutation, from a two-register table.
    const uint32_t c8B = 8u * B;
    const uint32_t msh = 1u << sh;  // q << sh == q * 2^sh
    const uint32_t kSel01 = 0x32143210u, kSel23 = 0x34563245u;  // byte selectors for nb = 0, 1 | 2, 3
    const uint32_t kPick = 0x10u + 0x22u * B;                   // picks table entry nb = B - lead
    const uint32_t m8 = opaque(0u - 8u);  // a multiplier the compiler cannot see: c = c8B - 8 l stays ONE multiply-add
#pragma unroll kUnroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t cb = (uint32_t)(codes >> (8 * j)) & 0xffu;
      const uint32_t l0 = cb & 3u, l1 = (cb >> 2) & 3u, l2 = (cb >> 4) & 3u, l3 = cb >> 6;
      const uint32_t c0 = mad_lo(l0, m8, c8B), c1 = mad_lo(l1, m8, c8B), c2 = mad_lo(l2, m8, c8B);  // 8 * stored bytes
      const uint32_t wi = pos >> 2, z = 8u * pos;  // the funnel shifts use z mod 32 = 8 * (pos & 3)
      const uint32_t A0 = img[wi], A1 = img[wi + 1], A2 = img[wi + 2], A3 = img[wi + 3];
      // at most 12 bytes per quad here: three words of string are enough
      const uint32_t S0 = __funnelshift_r(A0, A1, z), S1 = __funnelshift_r(A1, A2, z), S2 = __funnelshift_r(A2, A3, z);
      pos += 4u * B - (l0 + l1 + l2 + l3);
      const uint32_t U0 = __funnelshift_r(S0, S1, c0), U1 = __funnelshift_r(S1, S2, c0);
      const uint32_t X0 = __funnelshift_r(U0, U1, c1);
      const uint32_t X1 = __funnelshift_r(U1, S2 >> c0, c1);
      const uint32_t r3 = __funnelshift_r(X0, X1, c2);
      const uint32_t q0 = prmt(prev, S0, prmt(kSel01, kSel23, kPick - 0x22u * l0));
      const uint32_t q1 = prmt(q0, U0, prmt(kSel01, kSel23, kPick - 0x22u * l1));
      const uint32_t q2 = prmt(q1, X0, prmt(kSel01, kSel23, kPick - 0x22u * l2));
      const uint32_t q3 = prmt(q2, r3, prmt(kSel01, kSel23, kPick - 0x22u * l3));
      prev = q3;
      put(j, make_float4(__fadd_rn(__uint_as_float(q0 * msh), mu), __fadd_rn(__uint_as_float(q1 * msh), mu),
                         __fadd_rn(__uint_as_float(q2 * msh), mu), __fadd_rn(__uint_as_float(q3 * msh), mu)));
    }
    return true;
  }
  // General path (ragged slice, 4-byte field, lossless block): one out-of-line call per quad.
  DecodeCursor cur = {pos0, prev};
#pragma unroll kUnroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t cb = (uint32_t)(codes >> (8 * j)) & 0xffu;
    const uint32_t done = 4u * (uint32_t)j;
    put(j, decode_quad_generic(img, cur, cb, R, mu, lg.nv > done ? lg.nv - done : 0u));
  }
  return true;
}

// Ask L2 for the payload of group gp of the stream (a later CTA will stage it).  The two directory words
// are loaded by the caller early (dir_a, dir_e); nothing is validated here, a prefetch cannot fault.
__device__ __forceinline__ void prefetch_payload(const StreamView& sv, uint32_t dir_a, uint32_t dir_e) {
  if (dir_e <= dir_a || dir_e - dir_a > (uint32_t)kMaxGroupBytes / 4u || dir_e > sv.pw) return;
  const uint8_t* base = reinterpret_cast<const uint8_t*>(sv.words) + sv.base;
  for (uint32_t off = 4u * dir_a + 128u * threadIdx.x; off < 4u * dir_e; off += 128u * kThreads)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
}

// Stage group payload words [a, a+gw) of the stream into the image.  The copy starts at the 16-byte boundary
// at or below word a, so payload word j lands at img[(a & 3) + j] — decode_group reads the image through that
// shifted origin.  Where every 16-byte piece lies inside the stream (all groups but, at most, a stream's
// last), one thread hands the whole copy to the bulk-copy engine (`cp.async.bulk`, completion on `bar`): no
// load, no shared-memory store and no register passes through the lanes.  Returns true in that case: after
// the CTA's next barrier every thread waits with tma_wait_tile(bar).  Otherwise the words are copied by the
// lanes and the CTA's next barrier completes the staging.
__device__ __forceinline__ bool stage_payload(uint32_t* img, const StreamView& sv, uint64_t* bar) {
  const uint32_t shift = sv.a & 3u;
  const uint32_t start = sv.a - shift;                // aligned first word
  const uint32_t n_words = sv.gw + shift;             // words to bring in, from the aligned start
  const uint32_t n4 = (n_words + 3u) >> 2;            // 16-byte pieces
  const uint32_t* src = sv.words + (sv.base >> 2) + start;
  if (n4 != 0u && start + 4u * n4 <= sv.pw && (reinterpret_cast<uintptr_t>(src) & 15u) == 0u) {  // uniform
    if (threadIdx.x == 0) {
      const uint32_t b = smem_u32(bar), bytes = 16u * n4;
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_proxy_async();
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                       smem_u32(img)),
                   "l"(src), "r"(bytes), "r"(b)
                   : "memory");
    }
    return true;
  }
#pragma unroll 4
  for (uint32_t w = threadIdx.x; w < n_words; w += kThreads) img[w] = __ldcs(src + w);
  return false;
}

// ---------------------------------------------------------------------------------------------------
// kernels
// ---------------------------------------------------------------------------------------------------
// A group that cannot be encoded (corrupt input, a wait that ran out): report it, and publish poisoned size
// words so that no later group waits for this one.
__device__ __forceinline__ void give_up(const EncodeBatch& b, const JobGeom& jg, uint32_t g, uint32_t y, uint32_t code) {
  if (threadIdx.x != 0) return;
  raise(b.status, code);
  const SizeWords sw = size_words(b, y);
  st_relaxed_u64(&sw.A[g], pack_state(b.epoch, kFlagPoison, 0));
  if ((g & 31u) == 31u || g == jg.G - 1u) st_relaxed_u64(&sw.SA[g >> 5], pack_state(b.epoch, kFlagPoison, 0));
}

__global__ void __launch_bounds__(kThreads, 6) ccoll_compress_kernel(const __grid_constant__ EncodeBatch b) {
  Smem& sm = *reinterpret_cast<Smem*>(dyn_smem);
  uint8_t* rows = dyn_smem + kCtlBytes;
  const uint32_t g = blockIdx.x, y = blockIdx.y;
  grid_release();
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  uint8_t* sout = b.sout + (uint64_t)y * b.s_stride;
  if (jg.G == 0) {
    if (g == 0) write_empty_stream(b, y, sout);
    return;
  }
  if (g >= jg.G) return;
  const uint32_t rank = (uint32_t)((y + (uint32_t)b.rot) % (uint32_t)b.P);
  const float* x = b.x + (uint64_t)rank * b.x_rank_stride + jg.lo;
  const LaneGeom lg = lane_geom(jg, g);
  const bool tail = __any_sync(kFull, lg.nv != (uint32_t)kSliceVals);
  // (A TMA tile load into these rows was measured too: 78 us against 71 us.  Nothing else can run in this CTA
  // until its values are there, and the one bulk request comes back later than eight rounds of plain loads; in
  // the fused round the same tile load hides behind the staging of the payload and wins.)
  load_rows_padded_own(rows, x, jg, g);
  prefetch_group(x, jg, g + b.prefetch_distance);
  zero_image(sm.img);  // (this and the two words below are first used behind the barrier inside encode_group)
  if (threadIdx.x == 0) sm.prefix = 0u, sm.fail = 0u;
  __syncwarp();  // a warp reads only rows that it loaded itself
  if (tail) pad_ragged<PaddedRow>(rows, lg);
  float mx, mn;
  lane_minmax(make_row<PaddedRow>(rows, threadIdx.x), mx, mn);
  encode_group<PaddedRow>(sm, rows, lg, b, jg, g, y, sout, mx, mn, tail);
}

template <bool kDivide>
__global__ void __launch_bounds__(kThreads, 6) ccoll_reduce_kernel(const __grid_constant__ EncodeBatch b,
                                                                   const __grid_constant__ CUtensorMap x_map,
                                                                   const __grid_constant__ CUtensorMap sum_map) {
  Smem& sm = *reinterpret_cast<Smem*>(dyn_smem);
  uint8_t* rows = dyn_smem + kCtlBytes;
  const uint32_t g = blockIdx.x, y = blockIdx.y;
  grid_release();
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  uint8_t* sout = b.sout + (uint64_t)y * b.s_stride;
  if (jg.G == 0) {
    grid_acquire();
    if (g == 0) write_empty_stream(b, y, sout);
    return;
  }
  if (g >= jg.G) return;
  const uint32_t rank = (uint32_t)((y + (uint32_t)b.rot) % (uint32_t)b.P);
  const float* local = b.x + (uint64_t)rank * b.x_rank_stride + jg.lo;
  const LaneGeom lg = lane_geom(jg, g);
  TL(0);
  const bool tail = __any_sync(kFull, lg.nv != (uint32_t)kSliceVals);
  const PaddedRow row = make_row<PaddedRow>(rows, threadIdx.x);
  const bool whole = group_count(jg, g) == (uint32_t)kGroupValues;
  const bool tma = b.use_tma_in && whole;
  const uint32_t row0 = (jg.lo + g * (uint32_t)kGroupValues) >> 5;  // the group's first row in the rank buffer
  if (tma) {
    if (threadIdx.x == 0) tma_load_tile(&x_map, rows, &sm.bar, row0, b.x_rank_stride ? rank : 0u, kPaddedRowsBytes);
  } else {
    load_rows_padded(rows, local, jg, g);
  }
  prefetch_group(local, jg, g + b.prefetch_distance);
  if (threadIdx.x == 0) sm.prefix = 0u, sm.fail = 0u;

  // Everything above reads only this rank's own values, which no launch of a replay writes: in a replay this
  // grid may get here while the round before it is still draining.  Its streams are read from here on.
  grid_acquire();
  const uint8_t* sin = b.sin + (uint64_t)y * b.s_stride;
  const uint64_t in_bytes = b.sin_bytes ? b.sin_bytes[y] : b.sin_bytes_host;
  StreamView sv;
  float4 unused[8];
  float mx = __uint_as_float(0xff800000u), mn = __uint_as_float(0x7f800000u);  // -inf, +inf
  bool ok = open_group(sin, in_bytes, jg, g, sv);
  uint32_t nxt_a = 0u, nxt_e = 0u;  // directory entries of the group that will take over this SM slot
  if (ok && g + b.prefetch_distance < jg.G) {
    nxt_a = __ldg(sv.words + 8 + g + b.prefetch_distance);
    nxt_e = __ldg(sv.words + 8 + g + b.prefetch_distance + 1);
  }
  if (ok) {
    const bool bulk = stage_payload(sm.img, sv, &sm.bar_in);
    prefetch_payload(sv, nxt_a, nxt_e);
    __syncthreads();  // lane-copied words are in place; both mbarriers are initialised
    TL(1);
    if ((bulk && !tma_wait_tile(&sm.bar_in)) || (tma && !tma_wait_tile(&sm.bar))) {
      give_up(b, jg, g, y, kErrTimeout);
      return;
    }
    // decoded (op) local, one rounded operation per value, left in the lane's row
    ok = decode_group<true, kDivide, PaddedRow>(sm, sv, lg, min((uint32_t)kGroupBlocks, jg.nb - g * kGroupBlocks), unused, row,
                                     b.op, b.divisor, mx, mn);
  }
  TL(2);
  if (!ok) {  // a corrupt input
    if (tma && threadIdx.x == 0) tma_wait_tile(&sm.bar);  // the tile in flight must land before the CTA's memory goes
    give_up(b, jg, g, y, kErrCorrupt);
    return;
  }
  const bool tma_sum = b.sum_out && b.use_tma_sum && whole;
  if (tma_sum) fence_proxy_async();  // the results just written are about to be read by the TMA unit
  __syncthreads();  // every thread is done reading the incoming image (and has written its results)
  if (tma_sum && threadIdx.x == 0) tma_store_tile(&sum_map, rows, row0, b.sum_rank_stride ? rank : 0u);
  zero_image(sm.img);  // while the TMA unit reads the tile
  if (b.sum_out) {
    if (tma_sum) {
      if (threadIdx.x == 0) tma_store_wait();
    } else {
      store_rows_padded(rows, b.sum_out + (uint64_t)rank * b.sum_rank_stride + jg.lo, jg, g);
    }
    __syncthreads();  // the rows are about to be reused for staging
  }
  TL(3);
  if (tail) {
    pad_ragged<PaddedRow>(rows, lg);
    lane_minmax(row, mx, mn);
  }
  encode_group<PaddedRow>(sm, rows, lg, b, jg, g, y, sout, mx, mn, tail);
  TL(7);
}

// The incoming image is dead once every lane holds its decoded values in registers, so the rows the values
// leave through reuse the same shared memory: 18 KB per CTA, 12 CTAs per SM.  That occupancy caps the kernel
// at 40 registers and costs a few spilled words; measured, 12 CTAs with the spills (48 us on the 134 MB case)
// beat 9 CTAs without (50 us) now that the kernel waits on its bulk copy rather than on the load/store pipe.
__global__ void __launch_bounds__(kThreads, 12) ccoll_decode_kernel(const __grid_constant__ DecodeBatch b,
                                                                   const __grid_constant__ CUtensorMap out_map) {
  Smem& sm = *reinterpret_cast<Smem*>(dyn_smem);  // only sm.img is used here
  uint8_t* rows = dyn_smem;                        // aliases sm.img
  const uint32_t g = blockIdx.x, y = blockIdx.y, z = blockIdx.z;
  if (b.skip_mode == 1 && z == (y + (uint32_t)b.P - 1u) % (uint32_t)b.P) return;
  if (b.skip_mode == 2 && z == 0u) return;
  if (b.skip_mode == 3 && y == 0u) return;
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  if (g >= jg.G) return;
  const uint8_t* sin = b.sin + (uint64_t)y * b.s_stride;
  grid_acquire();
  const uint64_t in_bytes = b.sin_bytes ? b.sin_bytes[y] : b.sin_bytes_host;
  const uint32_t dest = b.skip_mode == 4 ? (y + (uint32_t)b.rot) % (uint32_t)b.P : z;
  float* out = b.scatter ? b.out + (uint64_t)y * b.out_rank_stride : b.out + (uint64_t)dest * b.out_rank_stride + jg.lo;
  const LaneGeom lg = lane_geom(jg, g);
  StreamView sv;
  float4 v[8];
  TL(0);
  bool ok = open_group(sin, in_bytes, jg, g, sv);
  TL(1);
  if (ok) {
    // (asking L2 for the payload of the group that will take over this SM slot pays in the fused kernel's
    // mix of loads, not here: 55.6 -> 54.2 us without it)
    uint64_t* bar = reinterpret_cast<uint64_t*>(dyn_smem + kDecodeBarOffset);  // behind the image and the rows
    const bool bulk = stage_payload(sm.img, sv, bar);
    __syncthreads();
    if (bulk && !tma_wait_tile(bar)) {
      if (threadIdx.x == 0) raise(b.status, kErrTimeout);
      return;
    }
    TL(2);
    float mx_unused, mn_unused;
    ok = decode_group<false>(sm, sv, lg, min((uint32_t)kGroupBlocks, jg.nb - g * kGroupBlocks), v, Row{nullptr, 0u}, 0,
                             0.0f, mx_unused, mn_unused);
  }
  if (!ok) {
    if (threadIdx.x == 0) raise(b.status, kErrCorrupt);
    return;
  }
  TL(3);
  __syncthreads();  // every lane is done reading the image
  {
    const Row row = row_of(rows, threadIdx.x);
#pragma unroll
    for (int j = 0; j < 8; ++j) row.set_quad(j, v[j]);
  }
  if (b.use_tma && group_count(jg, g) == (uint32_t)kGroupValues && (smem_u32(rows) & 1023u) == 0u) {
    // a complete group leaves as one tile: rows [first value / 32, +128) of the destination's plane
    fence_proxy_async();
    __syncthreads();
    TL(4);
    if (threadIdx.x == 0) {
      const uint32_t row0 = ((b.scatter ? 0u : jg.lo) + g * (uint32_t)kGroupValues) >> 5;
      tma_store_tile(&out_map, rows, row0, b.out_rank_stride ? (b.scatter ? y : dest) : 0u);
      tma_store_wait();
    }
  } else {
    __syncthreads();
    TL(4);
    store_rows(rows, out, jg, g);
  }
  TL(5);
}

}  // namespace

namespace {
constexpr int kSmemBytes = kCtlBytes + kPaddedRowsBytes;  // encoder and fused round: control block + padded rows
constexpr int kSmemCompress = kSmemBytes;
constexpr int kSmemDecode = kDecodeBarOffset + 16;

// Per device: opt in to the dynamic shared-memory size once, and learn how many CTAs of the encoding kernels
// are resident at a time (the distance of their L2 prefetch).
bool g_ready[64];
uint32_t g_slots[64];
// Tensor map of a buffer seen as [32 fp32][rows][planes] with 128-byte rows, tile = 32 x 128 x 1, 128-byte
// swizzle.  The encoder is a driver entry point looked up once through the runtime.  False if it cannot be
// had or refuses the arguments: the kernels then use their plain load/store paths.
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool make_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t planes, uint64_t plane_stride_bytes,
                   bool padded) {
  static EncodeTiledFn encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      fn = nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
  }();
  static const bool disabled = std::getenv("CCOLL_NO_TMA") != nullptr;  // forces the plain load/store paths (tests)
  if (disabled || !encode || (reinterpret_cast<uintptr_t>(base) & 15u)) return false;
  if (planes > 1 && ((plane_stride_bytes & 15u) || plane_stride_bytes >= (1ull << 40))) return false;
  const cuuint64_t dims[3] = {32u, rows, planes ? planes : 1u};
  const cuuint64_t strides[2] = {128u, planes > 1 ? plane_stride_bytes : 128u * rows};
  // padded: a box 36 values wide over rows of 32 -> shared-memory rows of 144 bytes, the last four values out of
  // bounds (zeros on a load, not written by a store); otherwise dense rows with the 128-byte swizzle
  const cuuint32_t box[3] = {padded ? (cuuint32_t)(kPaddedRowBytes / 4) : 32u, 128u, 1u};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, padded ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool device_ready() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (!g_ready[dev]) {
    int sms = 0, per_sm = 0;
    if (cudaFuncSetAttribute(ccoll_compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCompress) != cudaSuccess ||
        cudaFuncSetAttribute(ccoll_reduce_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(ccoll_reduce_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(ccoll_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemDecode) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ccoll_compress_kernel, kThreads, kSmemCompress) != cudaSuccess)
      return false;
    g_slots[dev] = (uint32_t)(sms * (per_sm > 0 ? per_sm : 1));
    g_ready[dev] = true;
  }
  return true;
}
}  // namespace

// Groups wait (bounded) on the sizes of earlier groups of their job; CTAs are issued in blockIdx order
// (x fastest), so the CTAs a group depends on are always resident or finished.
static EncodeBatch with_prefetch(const EncodeBatch& b, uint32_t jobs) {
  int dev = 0;
  cudaGetDevice(&dev);
  EncodeBatch c = b;
  // CTAs are issued x-fastest: with one job the slot of group g is taken over by group g + slots
  c.prefetch_distance = jobs == 1 ? g_slots[dev] : (g_slots[dev] + jobs - 1) / jobs;
  return c;
}
// The fp32 side of an encode batch as a tensor of 128-byte rows: [32 values][rows of a rank][ranks].
static bool rank_buffer_map(CUtensorMap* map, const float* base, uint64_t n, uint64_t rank_stride, int P) {
  std::memset(map, 0, sizeof(*map));
  return base && n / 32u >= 128u &&
         make_tile_map(map, base, n / 32u, rank_stride ? (uint64_t)P : 1u, rank_stride * 4u, /*padded=*/true);
}
// A launch that is being captured into a CUDA graph will run again with the epoch it was captured with, and
// would then take its own size words of the previous replay for fresh ones.  Such a launch gets a memset node
// in front of it that clears its size words (epoch 0 is never used), so every replay starts from "not written".
static bool is_capturing(cudaStream_t s) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &st) != cudaSuccess) {
    cudaGetLastError();  // e.g. the legacy stream while another stream captures: not a capture of this launch
    return false;
  }
  return st == cudaStreamCaptureStatusActive;
}
static bool clear_sizes(const EncodeBatch& b, uint32_t jobs, cudaStream_t s) {
  const size_t words = (size_t)jobs * b.state_stride;
  return words == 0 || cudaMemsetAsync(b.tile_state, 0, words * sizeof(uint64_t), s) == cudaSuccess;
}
bool launch_compress(const EncodeBatch& b0, uint32_t groups_x, uint32_t jobs, cudaStream_t s) {
  if (!device_ready() || (is_capturing(s) && !clear_sizes(b0, jobs, s))) return false;
  const EncodeBatch b = with_prefetch(b0, jobs);
  ccoll_compress_kernel<<<dim3(groups_x, jobs, 1), kThreads, kSmemCompress, s>>>(b);
  return true;
}
// With `behind_producer` the grid is launched with the programmatic-serialisation attribute: its CTAs may take
// the SM slots that the stream's previous grid (the producer of its input streams) leaves free while draining,
// run up to their grid_acquire() and wait there.
template <typename... Params, typename... Args>
static void launch_grid(void (*kernel)(Params...), dim3 grid, int smem, cudaStream_t s, bool behind_producer, Args&&... args) {
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  std::memset(&attr, 0, sizeof(attr));
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = behind_producer ? 1u : 0u;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
bool launch_reduce(const EncodeBatch& b0, uint32_t groups_x, uint32_t jobs, cudaStream_t s, bool behind_producer) {
  if (!device_ready()) return false;
  if (is_capturing(s)) {  // (captured launches are plain ones: the memset node sits between this grid and its producer)
    if (!clear_sizes(b0, jobs, s)) return false;
    behind_producer = false;
  }
  EncodeBatch b = with_prefetch(b0, jobs);
  CUtensorMap x_map, sum_map;
  b.use_tma_in = rank_buffer_map(&x_map, b.x, b.n, b.x_rank_stride, b.P) ? 1 : 0;
  b.use_tma_sum = rank_buffer_map(&sum_map, b.sum_out, b.n, b.sum_rank_stride, b.P) ? 1 : 0;
  launch_grid(b.op == 3 ? ccoll_reduce_kernel<true> : ccoll_reduce_kernel<false>, dim3(groups_x, jobs, 1), kSmemBytes, s,
              behind_producer, b, x_map, sum_map);
  return true;
}
bool launch_decode(const DecodeBatch& b0, uint32_t groups_x, uint32_t jobs, uint32_t ranks, cudaStream_t s,
                   bool behind_producer) {
  if (!device_ready()) return false;
  DecodeBatch b = b0;
  // The output as a tensor of 128-byte rows: [32 values][rows of a destination][destinations].
  CUtensorMap map;
  std::memset(&map, 0, sizeof(map));
  const uint64_t rows = (b.scatter ? b.chunk_len : b.n) / 32u;
  const uint64_t planes = b.out_rank_stride ? (b.scatter ? jobs : (b.skip_mode == 4 ? (uint32_t)b.P : ranks)) : 1u;
  b.use_tma = rows >= 128u && make_tile_map(&map, b.out, rows, planes, b.out_rank_stride * 4u, /*padded=*/false) ? 1 : 0;
  launch_grid(ccoll_decode_kernel, dim3(groups_x, jobs, ranks), kSmemDecode, s, behind_producer && !is_capturing(s), b, map);
  return true;
}

#ifdef CCOLL_TIMELINE
extern "C" int ccoll_debug_timeline(unsigned long long* host, size_t count) {
  return (int)cudaMemcpyFromSymbol(host, g_timeline, count * sizeof(unsigned long long));
}
#endif
}  // namespace ccoll
