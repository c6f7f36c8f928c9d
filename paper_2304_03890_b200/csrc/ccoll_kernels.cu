// ccoll_kernels.cu — device code of libccoll (see ccoll_kernels.cuh for the work decomposition and
// include/ccoll.h for the stream layout and the block rules).  Compiled with --fmad=false: every fp32
// operation of the block rules rounds once, exactly as stated.
#include "ccoll_kernels.cuh"

namespace ccoll {
namespace {

constexpr uint32_t kFull = 0xffffffffu;

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
// Warp-wide fp32 max / min in one instruction; a NaN in any lane makes the result NaN.
__device__ __forceinline__ float warp_max_nan(float v) {
  float r;
  asm volatile("redux.sync.max.NaN.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float warp_min_nan(float v) {
  float r;
  asm volatile("redux.sync.min.NaN.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t* p) {
  uint64_t v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u64(uint64_t* p, uint64_t v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
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

struct JobGeom {
  uint64_t lo;      // first value of the job inside the rank buffer
  uint64_t len;     // values in the job
  uint32_t nb;      // blocks
  uint32_t G;       // groups
  uint32_t m_last;  // values in the job's last block (1..128; 0 if the job is empty)
};
__device__ __forceinline__ JobGeom job_geom(uint64_t n, uint64_t C, uint32_t y) {
  JobGeom j;
  uint64_t lo = (uint64_t)y * C, hi = lo + C;
  j.lo = lo < n ? lo : n;
  hi = hi < n ? hi : n;
  j.len = hi - j.lo;
  j.nb = (uint32_t)((j.len + kL - 1) / kL);
  j.G = (j.nb + kGroupBlocks - 1) / kGroupBlocks;
  j.m_last = (uint32_t)(j.len - (uint64_t)(j.nb ? j.nb - 1 : 0) * kL);
  return j;
}

// ---------------------------------------------------------------------------------------------------
// shared memory
// ---------------------------------------------------------------------------------------------------
struct EncSmem {
  uint32_t img[kImgWords];   // payload image of the outgoing group (zeroed, filled by OR)
  uint32_t blk_mu[kGroupBlocks];
  uint32_t blk_R[kGroupBlocks];     // 0 = constant or absent block
  uint32_t blk_size[kGroupBlocks];  // record bytes, 0 = absent block
  uint32_t prefix;                  // exclusive prefix of this group, in words
  uint32_t fail;
};
struct DecSmem {
  uint32_t img[kImgWords];  // payload image of the incoming group
};

// ---------------------------------------------------------------------------------------------------
// encode side: one block (rules R1-R8), values of the lane in x0..x3
// ---------------------------------------------------------------------------------------------------
// Outputs: R (0 = constant), mu_bits, the lane's stored bytes as a little-endian 16-byte string W[0..3]
// (T bytes of it are meaningful), and the lane's lead-code byte.
template <bool kTail>
__device__ __forceinline__ void encode_block(float x0, float x1, float x2, float x3, uint32_t m, uint32_t lane,
                                             float eb, int eb_exp, uint32_t& mu_bits, uint32_t& R, uint32_t& W0,
                                             uint32_t& W1, uint32_t& W2, uint32_t& W3, uint32_t& T,
                                             uint32_t& code) {
  int nv = 4;
  if (kTail) {
    nv = (int)m - 4 * (int)lane;
    nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
    float f = __shfl_sync(kFull, x0, 0);  // element 0 always exists; it cannot change min or max
    if (nv < 1) x0 = f;
    if (nv < 2) x1 = f;
    if (nv < 3) x2 = f;
    if (nv < 4) x3 = f;
  }
  const float kInf = __uint_as_float(0x7f800000u);
  float mx = warp_max_nan(max_nan(max_nan(x0, x1), max_nan(x2, x3)));
  float mn = warp_min_nan(min_nan(min_nan(x0, x1), min_nan(x2, x3)));
  bool special = !(fabsf(mx) < kInf) || !(fabsf(mn) < kInf);  // NaN or Inf somewhere in the block
  float mu = __fadd_rn(__fmul_rn(0.5f, mn), __fmul_rn(0.5f, mx));
  uint32_t mub = __float_as_uint(mu);
  if ((mub << 1) == 0u) mub = 0u;  // a zero of either sign becomes +0
  mu = __uint_as_float(mub);
  float r = fmaxf(__fsub_rn(mx, mu), __fsub_rn(mu, mn));
  W0 = W1 = W2 = W3 = 0u;
  T = 0u;
  code = 0u;
  if (!special && r <= eb) {
    R = 0u;
    mu_bits = mub;
    return;
  }
  int m_bits = (int)((__float_as_uint(r) >> 23) & 0xffu) - eb_exp + 1;
  bool lossless = special || m_bits >= 23;
  R = lossless ? 32u : (uint32_t)(9 + m_bits);
  if (lossless) {
    mub = 0u;
    mu = 0.0f;
  }
  mu_bits = mub;
  uint32_t sh = 32u - R;
  uint32_t q0 = __float_as_uint(lossless ? x0 : __fsub_rn(x0, mu)) >> sh;
  uint32_t q1 = __float_as_uint(lossless ? x1 : __fsub_rn(x1, mu)) >> sh;
  uint32_t q2 = __float_as_uint(lossless ? x2 : __fsub_rn(x2, mu)) >> sh;
  uint32_t q3 = __float_as_uint(lossless ? x3 : __fsub_rn(x3, mu)) >> sh;
  uint32_t B = (R + 7u) >> 3;
  uint32_t min_nb = (B == 4u) ? 1u : 0u;  // lead is capped at 3, so a 4-byte field always stores a byte
  uint32_t p0 = __shfl_up_sync(kFull, q3, 1);
  if (lane == 0) p0 = 0u;
  // stored bytes of an element = significant bytes of (q xor predecessor)
  uint32_t nb0 = max((39u - (uint32_t)__clz(q0 ^ p0)) >> 3, min_nb);
  uint32_t nb1 = max((39u - (uint32_t)__clz(q1 ^ q0)) >> 3, min_nb);
  uint32_t nb2 = max((39u - (uint32_t)__clz(q2 ^ q1)) >> 3, min_nb);
  uint32_t nb3 = max((39u - (uint32_t)__clz(q3 ^ q2)) >> 3, min_nb);
  if (kTail) {
    uint32_t l0 = B - nb0, l1 = B - nb1, l2 = B - nb2, l3 = B - nb3;
    if (nv < 1) nb0 = 0u, l0 = 0u;
    if (nv < 2) nb1 = 0u, l1 = 0u;
    if (nv < 3) nb2 = 0u, l2 = 0u;
    if (nv < 4) nb3 = 0u, l3 = 0u;
    code = l0 | (l1 << 2) | (l2 << 4) | (l3 << 6);
  } else {
    code = B * 0x55u - (nb0 + 4u * nb1 + 16u * nb2 + 64u * nb3);
  }
  T = nb0 + nb1 + nb2 + nb3;
  // the low nb bytes of q, most significant first, as a little-endian integer
  uint32_t e0 = __funnelshift_rc(__byte_perm(q0, 0u, 0x0123), 0u, 32u - 8u * nb0);
  uint32_t e1 = __funnelshift_rc(__byte_perm(q1, 0u, 0x0123), 0u, 32u - 8u * nb1);
  uint32_t e2 = __funnelshift_rc(__byte_perm(q2, 0u, 0x0123), 0u, 32u - 8u * nb2);
  uint32_t e3 = __funnelshift_rc(__byte_perm(q3, 0u, 0x0123), 0u, 32u - 8u * nb3);
  uint32_t s0 = 8u * nb0, s2 = 8u * nb2;
  uint32_t lo01 = e0 | __funnelshift_lc(0u, e1, s0), hi01 = __funnelshift_lc(e1, 0u, s0);
  uint32_t lo23 = e2 | __funnelshift_lc(0u, e3, s2), hi23 = __funnelshift_lc(e3, 0u, s2);
  uint32_t s = 8u * (nb0 + nb1);
  bool upper = s >= 32u;
  uint32_t a = upper ? s - 32u : s;
  uint32_t t0 = __funnelshift_lc(0u, lo23, a), t1 = __funnelshift_lc(lo23, hi23, a),
           t2 = __funnelshift_lc(hi23, 0u, a);
  W0 = upper ? lo01 : (lo01 | t0);
  W1 = upper ? (hi01 | t0) : (hi01 | t1);
  W2 = upper ? t1 : t2;
  W3 = upper ? t2 : 0u;
}

// The image is zeroed once and then filled ONLY by atomic OR, so bytes of one word may come from any lane.
__device__ __forceinline__ void or_byte(uint32_t* img, uint32_t off, uint32_t byte) {
  atomicOr(&img[off >> 2], (byte & 0xffu) << (8u * (off & 3u)));
}

// OR a lane's T-byte string into the image at byte offset off.
__device__ __forceinline__ void place_string(uint32_t* img, uint32_t off, uint32_t T, uint32_t W0, uint32_t W1,
                                             uint32_t W2, uint32_t W3) {
  uint32_t z = 8u * (off & 3u);
  uint32_t wi = off >> 2;
  uint32_t cnt = ((off & 3u) + T + 3u) >> 2;
  uint32_t V0 = W0 << z;
  uint32_t V1 = __funnelshift_l(W0, W1, z);
  uint32_t V2 = __funnelshift_l(W1, W2, z);
  uint32_t V3 = __funnelshift_l(W2, W3, z);
  uint32_t V4 = __funnelshift_l(W3, 0u, z);
  if (cnt > 0) atomicOr(&img[wi], V0);
  if (cnt > 1) atomicOr(&img[wi + 1], V1);
  if (cnt > 2) atomicOr(&img[wi + 2], V2);
  if (cnt > 3) atomicOr(&img[wi + 3], V3);
  if (cnt > 4) atomicOr(&img[wi + 4], V4);
}

// inclusive warp scan of three 10-bit fields packed in one word
__device__ __forceinline__ uint32_t warp_scan_packed(uint32_t v, uint32_t lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t t = __shfl_up_sync(kFull, v, d);
    if (lane >= (uint32_t)d) v += t;
  }
  return v;
}
__device__ __forceinline__ uint32_t warp_scan_u32(uint32_t v, uint32_t lane) { return warp_scan_packed(v, lane); }

// Decoupled look-back over the groups of one job (tile order = blockIdx.x order, which is the order CTAs
// are issued in).  Called by all lanes of warp 0.  Returns false if it gave up; every wait is bounded.
__device__ __forceinline__ bool lookback(uint64_t* state, uint32_t g, uint32_t words, uint32_t epoch,
                                         uint32_t lane, uint32_t* status, uint32_t& excl_out) {
  if (g == 0) {
    if (lane == 0) st_relaxed_u64(&state[0], pack_state(epoch, kFlagPrefix, words));
    excl_out = 0;
    return true;
  }
  if (lane == 0) st_relaxed_u64(&state[g], pack_state(epoch, kFlagAggregate, words));
  uint32_t excl = 0;
  int base = (int)g - 1;
  uint32_t spins = 0;
  bool ok = true;
  while (true) {
    int t = base - (int)lane;
    uint32_t flag = kFlagPrefix, value = 0;  // tiles before the first one: an empty prefix
    if (t >= 0) {
      uint64_t w = ld_relaxed_u64(&state[t]);
      flag = ((uint32_t)(w >> 32) == epoch) ? (uint32_t)(w >> 30) & 3u : 0u;
      value = (uint32_t)w & kValueMask;
    }
    uint32_t ready = __ballot_sync(kFull, flag != 0u);
    uint32_t closed = __ballot_sync(kFull, flag == kFlagPrefix || flag == kFlagPoison);
    uint32_t first = closed ? (uint32_t)__ffs(closed) - 1u : 32u;
    uint32_t need = (first >= 31u) ? kFull : ((2u << first) - 1u);
    if ((ready & need) == need) {
      uint32_t poison = __ballot_sync(kFull, flag == kFlagPoison) & need;
      uint32_t v = ((need >> lane) & 1u) ? value : 0u;
      excl += __reduce_add_sync(kFull, v);
      if (poison) {
        ok = false;
        break;
      }
      if (first != 32u) break;
      base -= 32;
      continue;
    }
    if (++spins > kSpinLimit) {
      ok = false;
      if (lane == 0) raise(status, kErrTimeout);
      break;
    }
    __nanosleep(64);
  }
  if (lane == 0)
    st_relaxed_u64(&state[g], ok ? pack_state(epoch, kFlagPrefix, excl + words) : pack_state(epoch, kFlagPoison, 0));
  excl_out = excl;
  return ok;
}

// Encode the 8 blocks a warp holds in v[], build the group image, find the group's place in the stream
// and copy it out.  cnt = blocks this warp owns in the group; nblk = blocks in the group.
__device__ __forceinline__ void encode_group(EncSmem& sm, float4 (&v)[kWarpBlocks], const EncodeBatch& b,
                                             const JobGeom& jg, uint32_t g, uint32_t y, uint8_t* sout) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nblk = min((uint32_t)kGroupBlocks, jg.nb - g * kGroupBlocks);
  const int cnt = max(0, min(kWarpBlocks, (int)nblk - (int)(warp * kWarpBlocks)));
  const uint32_t last_blk = jg.nb - 1 - g * kGroupBlocks;  // group-relative index of the job's last block

  uint32_t W[kWarpBlocks][4];
  uint32_t tp[3] = {0u, 0u, 0u};  // per-lane stored-byte counts of the 8 blocks, three 10-bit fields per word
  uint32_t codes[2] = {0u, 0u};   // per-lane lead-code bytes of the 8 blocks
  uint32_t R_mine = 0u, mu_mine = 0u;  // lane i keeps R and mu of the warp's block i
#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    W[i][0] = W[i][1] = W[i][2] = W[i][3] = 0u;
    if (i < cnt) {
      uint32_t blk = warp * kWarpBlocks + i;
      uint32_t mu_bits, R, T, code;
      if (blk == last_blk && jg.m_last != (uint32_t)kL)
        encode_block<true>(v[i].x, v[i].y, v[i].z, v[i].w, jg.m_last, lane, b.eb, b.eb_exp, mu_bits, R, W[i][0],
                           W[i][1], W[i][2], W[i][3], T, code);
      else
        encode_block<false>(v[i].x, v[i].y, v[i].z, v[i].w, kL, lane, b.eb, b.eb_exp, mu_bits, R, W[i][0], W[i][1],
                            W[i][2], W[i][3], T, code);
      tp[i / 3] |= T << (10 * (i % 3));
      codes[i / 4] |= code << (8 * (i % 4));
      if (lane == (uint32_t)i) {
        R_mine = R;
        mu_mine = mu_bits;
      }
    }
  }
  // exclusive offsets of every lane's bytes inside its block's record, and the records' sizes
  uint32_t incl[3], tot[3];
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    incl[k] = warp_scan_packed(tp[k], lane);
    tot[k] = __shfl_sync(kFull, incl[k], 31);
  }
  if (lane < (uint32_t)kWarpBlocks) {
    uint32_t blk = warp * kWarpBlocks + lane;
    uint32_t size = 0u;
    if ((int)lane < cnt) {
      uint32_t total = (tot[lane / 3] >> (10 * (lane % 3))) & 0x3ffu;
      uint32_t m = (blk == last_blk) ? jg.m_last : (uint32_t)kL;
      size = R_mine ? 5u + ((m + 3u) >> 2) + total : 4u;
    }
    sm.blk_mu[blk] = mu_mine;
    sm.blk_R[blk] = R_mine;
    sm.blk_size[blk] = size;
  }
  __syncthreads();  // also orders the zero-fill of the image before the ORs below

  // every warp derives the offsets of all 32 records (cheap, and saves a barrier)
  uint32_t my_size = sm.blk_size[lane];
  uint32_t my_R = sm.blk_R[lane];
  uint32_t bitmap = __ballot_sync(kFull, my_R != 0u);
  uint32_t k = (uint32_t)__popc(bitmap);
  uint32_t incl_sz = warp_scan_u32(my_size, lane);
  uint32_t my_off = 2u * k + incl_sz - my_size;
  uint32_t raw = 2u * k + __shfl_sync(kFull, incl_sz, 31);
  uint32_t words = (raw + 3u) >> 2;

  if (warp == 0) {
    if (my_R != 0u) {
      uint32_t rank = (uint32_t)__popc(bitmap & ((1u << lane) - 1u));
      atomicOr(&sm.img[rank >> 1], my_size << (16u * (rank & 1u)));
    }
  }
#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    if (i < cnt) {
      uint32_t blk = warp * kWarpBlocks + i;
      uint32_t off = __shfl_sync(kFull, my_off, blk);
      uint32_t R = sm.blk_R[blk];
      uint32_t mu_bits = sm.blk_mu[blk];
      if (R == 0u) {
        if (lane < 4u) or_byte(sm.img, off + lane, mu_bits >> (8u * lane));
      } else {
        uint32_t m = (blk == last_blk) ? jg.m_last : (uint32_t)kL;
        uint32_t cb = (m + 3u) >> 2;
        if (lane < 5u) or_byte(sm.img, off + lane, (lane < 4u) ? (mu_bits >> (8u * lane)) : R);
        if (lane < cb) or_byte(sm.img, off + 5u + lane, codes[i / 4] >> (8 * (i % 4)));
        uint32_t T = (tp[i / 3] >> (10 * (i % 3))) & 0x3ffu;
        uint32_t excl = ((incl[i / 3] >> (10 * (i % 3))) & 0x3ffu) - T;
        place_string(sm.img, off + 5u + cb + excl, T, W[i][0], W[i][1], W[i][2], W[i][3]);
      }
    }
  }

  // place of the group in the stream
  if (warp == 0) {
    uint32_t excl;
    bool ok = lookback(b.tile_state + (uint64_t)y * b.tiles_per_job, g, words, b.epoch, lane, b.status, excl);
    if (lane == 0) {
      sm.prefix = excl;
      sm.fail = ok ? 0u : 1u;
    }
  }
  __syncthreads();
  const uint32_t prefix = sm.prefix;
  if (sm.fail) return;
  const uint32_t base = payload_base(jg.G);
  const uint64_t end = (uint64_t)base + 4ull * ((uint64_t)prefix + words);
  uint32_t* out32 = reinterpret_cast<uint32_t*>(sout);
  if (end > b.out_cap) {
    if (tid == 0) raise(b.status, kErrCapacity);
    return;
  }
  uint32_t* dst = out32 + (base >> 2) + prefix;
  for (uint32_t j = tid; j < words; j += kThreads) dst[j] = sm.img[j];
  if (tid == 0) {
    out32[8 + g] = prefix;                 // dir[g]
    out32[8 + jg.G + 1 + g] = bitmap;      // bitmap[g]
  }
  if (g == 0 && tid >= 32 && tid < 32 + 4) {
    // static part of the header and the zero pad between the bitmap and the payload
    uint32_t t = tid - 32;
    if (t == 0) {
      out32[0] = kMagic;
      out32[1] = 0u;
      out32[2] = (uint32_t)jg.len;
      out32[3] = (uint32_t)(jg.len >> 32);
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

__device__ __forceinline__ void zero_image(uint32_t* img) {
  uint4* p = reinterpret_cast<uint4*>(img);
  for (uint32_t j = threadIdx.x; j < (uint32_t)kImgWords / 4; j += kThreads) p[j] = make_uint4(0u, 0u, 0u, 0u);
}

// Load the (up to) 8 blocks a warp owns: one 128-bit streaming load per lane and block.
__device__ __forceinline__ void load_blocks(const float* x, const JobGeom& jg, uint32_t g, float4 (&v)[kWarpBlocks]) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    uint32_t gblk = g * kGroupBlocks + warp * kWarpBlocks + i;
    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (gblk < jg.nb) {
      const float* p = x + (uint64_t)gblk * kL + 4u * lane;
      uint32_t m = (gblk == jg.nb - 1) ? jg.m_last : (uint32_t)kL;
      if (4u * lane + 4u <= m) {
        v[i] = __ldcs(reinterpret_cast<const float4*>(p));
      } else {
        if (4u * lane + 0u < m) v[i].x = __ldcs(p + 0);
        if (4u * lane + 1u < m) v[i].y = __ldcs(p + 1);
        if (4u * lane + 2u < m) v[i].z = __ldcs(p + 2);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// decode side
// ---------------------------------------------------------------------------------------------------
struct StreamView {
  const uint32_t* words;  // the stream as 32-bit words
  uint32_t G, base;       // groups, payload_base
  uint32_t a, gw, map;    // first payload word of the group, its length in words, its bitmap
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
  return true;
}

// Decode the blocks this warp owns in group g into v[].  Returns false (for the whole CTA) on a corrupt group.
__device__ __forceinline__ bool decode_group(DecSmem& sm, const StreamView& sv, const JobGeom& jg, uint32_t g,
                                             float4 (&v)[kWarpBlocks]) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nblk = min((uint32_t)kGroupBlocks, jg.nb - g * kGroupBlocks);
  const int cnt = max(0, min(kWarpBlocks, (int)nblk - (int)(warp * kWarpBlocks)));
  const uint32_t last_blk = jg.nb - 1 - g * kGroupBlocks;

  // stage the group's payload in shared memory
  const uint32_t* src = sv.words + (sv.base >> 2) + sv.a;
  for (uint32_t j = tid; j < sv.gw; j += kThreads) sm.img[j] = __ldcs(src + j);
  __syncthreads();

  // offsets of the 32 records: lane b looks at block b
  bool bad = false;
  const uint32_t map = sv.map;
  const uint32_t k = (uint32_t)__popc(map);
  uint32_t my_size = 0u;
  if (lane < nblk) {
    if ((map >> lane) & 1u) {
      uint32_t rank = (uint32_t)__popc(map & ((1u << lane) - 1u));
      my_size = (rank < 2u * sv.gw) ? reinterpret_cast<const uint16_t*>(sm.img)[rank] : 0u;
    } else {
      my_size = 4u;
    }
  }
  uint32_t incl_sz = warp_scan_u32(my_size, lane);
  uint32_t my_off = 2u * k + incl_sz - my_size;
  uint32_t raw = 2u * k + __shfl_sync(kFull, incl_sz, 31);
  if (((raw + 3u) >> 2) != sv.gw) bad = true;

  // headers and lead codes of this warp's blocks, then one packed scan for all of them
  uint32_t tp[3] = {0u, 0u, 0u};
  uint32_t codes[2] = {0u, 0u};
  if (!bad) {
#pragma unroll
    for (int i = 0; i < kWarpBlocks; ++i) {
      if (i < cnt) {
        uint32_t blk = warp * kWarpBlocks + i;
        if ((map >> blk) & 1u) {
          uint32_t off = __shfl_sync(kFull, my_off, blk);
          uint32_t R = img_u8(sm.img, off + 4u);
          uint32_t B = (R + 7u) >> 3;
          if (!((R >= 10u && R <= 32u))) bad = true;
          uint32_t m = (blk == last_blk) ? jg.m_last : (uint32_t)kL;
          uint32_t cb = (m + 3u) >> 2;
          uint32_t code = (lane < cb && !bad) ? img_u8(sm.img, off + 5u + lane) : 0u;
          int nv = (int)m - 4 * (int)lane;
          nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
          uint32_t T = 0u;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t lead = (code >> (2 * j)) & 3u;
            if (j < nv) {
              if (lead > B) bad = true;
              T += B - lead;
            } else if (lead) {
              bad = true;
            }
          }
          if (bad) T = 0u;
          tp[i / 3] |= (T & 0x3ffu) << (10 * (i % 3));
          codes[i / 4] |= code << (8 * (i % 4));
        }
      }
    }
  }
  bad = __any_sync(kFull, bad);
  uint32_t incl[3], tot[3];
#pragma unroll
  for (int kk = 0; kk < 3; ++kk) {
    incl[kk] = warp_scan_packed(tp[kk], lane);
    tot[kk] = __shfl_sync(kFull, incl[kk], 31);
  }
  if (!bad) {
#pragma unroll
    for (int i = 0; i < kWarpBlocks; ++i) {
      if (i < cnt) {
        uint32_t blk = warp * kWarpBlocks + i;
        if ((map >> blk) & 1u) {
          uint32_t m = (blk == last_blk) ? jg.m_last : (uint32_t)kL;
          uint32_t size = __shfl_sync(kFull, my_size, blk);
          uint32_t total = (tot[i / 3] >> (10 * (i % 3))) & 0x3ffu;
          if (size != 5u + ((m + 3u) >> 2) + total) bad = true;
        }
      }
    }
  }
  if (__syncthreads_or(bad ? 1 : 0)) return false;

#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < cnt) {
      uint32_t blk = warp * kWarpBlocks + i;
      uint32_t off = __shfl_sync(kFull, my_off, blk);
      uint32_t mu_bits = img_u32(sm.img, off);
      float mu = __uint_as_float(mu_bits);
      if (!((map >> blk) & 1u)) {
        v[i] = make_float4(mu, mu, mu, mu);
      } else {
        uint32_t R = img_u8(sm.img, off + 4u);
        uint32_t B = (R + 7u) >> 3;
        uint32_t m = (blk == last_blk) ? jg.m_last : (uint32_t)kL;
        uint32_t cb = (m + 3u) >> 2;
        uint32_t code = (codes[i / 4] >> (8 * (i % 4))) & 0xffu;
        int nv = (int)m - 4 * (int)lane;
        nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
        uint32_t nb0 = nv > 0 ? B - (code & 3u) : 0u;
        uint32_t nb1 = nv > 1 ? B - ((code >> 2) & 3u) : 0u;
        uint32_t nb2 = nv > 2 ? B - ((code >> 4) & 3u) : 0u;
        uint32_t nb3 = nv > 3 ? B - ((code >> 6) & 3u) : 0u;
        uint32_t T = (tp[i / 3] >> (10 * (i % 3))) & 0x3ffu;
        uint32_t excl = ((incl[i / 3] >> (10 * (i % 3))) & 0x3ffu) - T;
        // the lane's stored bytes as a little-endian 16-byte string
        uint32_t so = off + 5u + cb + excl;
        uint32_t wi = so >> 2, z = 8u * (so & 3u);
        uint32_t A0 = sm.img[wi], A1 = sm.img[wi + 1], A2 = sm.img[wi + 2], A3 = sm.img[wi + 3], A4 = sm.img[wi + 4];
        uint32_t S0 = __funnelshift_r(A0, A1, z), S1 = __funnelshift_r(A1, A2, z), S2 = __funnelshift_r(A2, A3, z),
                 S3 = __funnelshift_r(A3, A4, z);
        // peel the four elements off the front of the string
        uint32_t r0 = S0;
        uint32_t c0 = 8u * nb0;
        uint32_t U0 = __funnelshift_rc(S0, S1, c0), U1 = __funnelshift_rc(S1, S2, c0), U2 = __funnelshift_rc(S2, S3, c0);
        uint32_t r1 = U0;
        uint32_t c1 = 8u * nb1;
        uint32_t X0 = __funnelshift_rc(U0, U1, c1), X1 = __funnelshift_rc(U1, U2, c1);
        uint32_t r2 = X0;
        uint32_t r3 = __funnelshift_rc(X0, X1, 8u * nb2);
        // stored bytes as a right-aligned big-endian value, and the byte mask they cover
        uint32_t v0 = __funnelshift_rc(__byte_perm(r0, 0u, 0x0123), 0u, 32u - 8u * nb0);
        uint32_t v1 = __funnelshift_rc(__byte_perm(r1, 0u, 0x0123), 0u, 32u - 8u * nb1);
        uint32_t v2 = __funnelshift_rc(__byte_perm(r2, 0u, 0x0123), 0u, 32u - 8u * nb2);
        uint32_t v3 = __funnelshift_rc(__byte_perm(r3, 0u, 0x0123), 0u, 32u - 8u * nb3);
        uint32_t m0 = __funnelshift_rc(kFull, 0u, 32u - 8u * nb0);
        uint32_t m1 = __funnelshift_rc(kFull, 0u, 32u - 8u * nb1);
        uint32_t m2 = __funnelshift_rc(kFull, 0u, 32u - 8u * nb2);
        uint32_t m3 = __funnelshift_rc(kFull, 0u, 32u - 8u * nb3);
        // resolve the elided leading bytes inside the lane as if nothing came from the left ...
        uint32_t l0 = v0;
        uint32_t l1 = v1 | (l0 & ~m1);
        uint32_t l2 = v2 | (l1 & ~m2);
        uint32_t l3 = v3 | (l2 & ~m3);
        uint32_t k0 = m0, k1 = k0 | m1, k2 = k1 | m2, k3 = k2 | m3;
        // ... then carry the last code across lanes: bytes a lane does not cover come from its left
        uint32_t cv = l3, cm = k3;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          uint32_t tv = __shfl_up_sync(kFull, cv, d);
          uint32_t tm = __shfl_up_sync(kFull, cm, d);
          cv = cv | (tv & ~cm);
          cm = cm | tm;
        }
        uint32_t carry = __shfl_up_sync(kFull, cv, 1);
        if (lane == 0) carry = 0u;
        uint32_t q0 = l0 | (carry & ~k0), q1 = l1 | (carry & ~k1), q2 = l2 | (carry & ~k2), q3 = l3 | (carry & ~k3);
        if (R == 32u) {
          v[i] = make_float4(__uint_as_float(q0), __uint_as_float(q1), __uint_as_float(q2), __uint_as_float(q3));
        } else {
          uint32_t sh = 32u - R;
          v[i] = make_float4(__fadd_rn(__uint_as_float(q0 << sh), mu), __fadd_rn(__uint_as_float(q1 << sh), mu),
                             __fadd_rn(__uint_as_float(q2 << sh), mu), __fadd_rn(__uint_as_float(q3 << sh), mu));
        }
      }
    }
  }
  return true;
}

// Store the blocks a warp decoded (or summed): one 128-bit store per lane and block.
__device__ __forceinline__ void store_blocks(float* out, const JobGeom& jg, uint32_t g, const float4 (&v)[kWarpBlocks]) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    uint32_t gblk = g * kGroupBlocks + warp * kWarpBlocks + i;
    if (gblk < jg.nb) {
      float* p = out + (uint64_t)gblk * kL + 4u * lane;
      uint32_t m = (gblk == jg.nb - 1) ? jg.m_last : (uint32_t)kL;
      if (4u * lane + 4u <= m) {
        __stcs(reinterpret_cast<float4*>(p), v[i]);
      } else {
        if (4u * lane + 0u < m) p[0] = v[i].x;
        if (4u * lane + 1u < m) p[1] = v[i].y;
        if (4u * lane + 2u < m) p[2] = v[i].z;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// kernels
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) compress_kernel(const __grid_constant__ EncodeBatch b) {
  __shared__ __align__(16) EncSmem sm;
  const uint32_t g = blockIdx.x, y = blockIdx.y;
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  uint8_t* sout = b.sout + (uint64_t)y * b.s_stride;
  if (jg.G == 0) {
    if (g == 0) write_empty_stream(b, y, sout);
    return;
  }
  if (g >= jg.G) return;
  const uint32_t rank = (uint32_t)((y + (uint32_t)b.rot) % (uint32_t)b.P);
  const float* x = b.x + (uint64_t)rank * b.x_rank_stride + jg.lo;
  float4 v[kWarpBlocks];
  load_blocks(x, jg, g, v);
  zero_image(sm.img);
  encode_group(sm, v, b, jg, g, y, sout);
}

__global__ void __launch_bounds__(kThreads) reduce_kernel(const __grid_constant__ EncodeBatch b) {
  __shared__ __align__(16) EncSmem sm;
  __shared__ __align__(16) DecSmem dm;
  const uint32_t g = blockIdx.x, y = blockIdx.y;
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  uint8_t* sout = b.sout + (uint64_t)y * b.s_stride;
  if (jg.G == 0) {
    if (g == 0) write_empty_stream(b, y, sout);
    return;
  }
  if (g >= jg.G) return;
  const uint32_t rank = (uint32_t)((y + (uint32_t)b.rot) % (uint32_t)b.P);
  const float* local = b.x + (uint64_t)rank * b.x_rank_stride + jg.lo;
  float4 loc[kWarpBlocks];
  load_blocks(local, jg, g, loc);
  zero_image(sm.img);
  const uint8_t* sin = b.sin + (uint64_t)y * b.s_stride;
  const uint64_t in_bytes = b.sin_bytes ? b.sin_bytes[y] : b.sin_bytes_host;
  StreamView sv;
  float4 v[kWarpBlocks];
  bool ok = open_group(sin, in_bytes, jg, g, sv);
  if (ok) ok = decode_group(dm, sv, jg, g, v);
  if (!ok) {
    // a corrupt input: report it, and keep the look-back chain alive with a poisoned entry
    if (threadIdx.x == 0) {
      raise(b.status, kErrCorrupt);
      st_relaxed_u64(b.tile_state + (uint64_t)y * b.tiles_per_job + g, pack_state(b.epoch, kFlagPoison, 0));
    }
    return;
  }
#pragma unroll
  for (int i = 0; i < kWarpBlocks; ++i) {
    v[i].x = __fadd_rn(v[i].x, loc[i].x);
    v[i].y = __fadd_rn(v[i].y, loc[i].y);
    v[i].z = __fadd_rn(v[i].z, loc[i].z);
    v[i].w = __fadd_rn(v[i].w, loc[i].w);
  }
  if (b.sum_out) store_blocks(b.sum_out + (uint64_t)rank * b.sum_rank_stride + jg.lo, jg, g, v);
  encode_group(sm, v, b, jg, g, y, sout);
}

__global__ void __launch_bounds__(kThreads) decode_kernel(const __grid_constant__ DecodeBatch b) {
  __shared__ __align__(16) DecSmem dm;
  const uint32_t g = blockIdx.x, y = blockIdx.y, z = blockIdx.z;
  if (b.skip_mode == 1 && z == (y + (uint32_t)b.P - 1u) % (uint32_t)b.P) return;
  if (b.skip_mode == 2 && z == 0u) return;
  if (b.skip_mode == 3 && y == 0u) return;
  const JobGeom jg = job_geom(b.n, b.chunk_len, y);
  if (g >= jg.G) return;
  const uint8_t* sin = b.sin + (uint64_t)y * b.s_stride;
  const uint64_t in_bytes = b.sin_bytes ? b.sin_bytes[y] : b.sin_bytes_host;
  float* out = b.scatter ? b.out + (uint64_t)y * b.out_rank_stride : b.out + (uint64_t)z * b.out_rank_stride + jg.lo;
  StreamView sv;
  float4 v[kWarpBlocks];
  bool ok = open_group(sin, in_bytes, jg, g, sv);
  if (ok) ok = decode_group(dm, sv, jg, g, v);
  if (!ok) {
    if (threadIdx.x == 0) raise(b.status, kErrCorrupt);
    return;
  }
  store_blocks(out, jg, g, v);
}

}  // namespace

void launch_compress(const EncodeBatch& b, uint32_t groups_x, uint32_t jobs, cudaStream_t s) {
  compress_kernel<<<dim3(groups_x, jobs, 1), kThreads, 0, s>>>(b);
}
void launch_reduce(const EncodeBatch& b, uint32_t groups_x, uint32_t jobs, cudaStream_t s) {
  reduce_kernel<<<dim3(groups_x, jobs, 1), kThreads, 0, s>>>(b);
}
void launch_decode(const DecodeBatch& b, uint32_t groups_x, uint32_t jobs, uint32_t ranks, cudaStream_t s) {
  decode_kernel<<<dim3(groups_x, jobs, ranks), kThreads, 0, s>>>(b);
}

}  // namespace ccoll
