// Device-side helpers: ordered float keys, bf16 MMA, streaming loads, the indexer score core.
#pragma once

#include "rtp_internal.cuh"

namespace rtp {

// ---- ordered keys: unsigned comparison of okey(a), okey(b) == float comparison of a, b ----------
__device__ __forceinline__ uint32_t okey(float s) {
  uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float okey_to_float(uint32_t k) {
  uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(b);
}

__device__ __forceinline__ void set_status(int32_t* status, int code) {
  if (status) atomicMax(status, code);
}

// ---- streaming 16-byte load (read-only data that is not reused by this SM) -----------------------
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld_stream_v2(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// ---- warp MMA m16n8k16, bf16 inputs, fp32 accumulate ------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1, const float (&c)[4]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%10,%11,%12,%13};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// ---- indexer score core --------------------------------------------------------------------------
// One warp scores 16 consecutive index keys (512 contiguous bytes, one 16-byte load per lane)
// against up to 16 projected queries held as an MMA A fragment.  The 16 index dimensions are
// fed to the MMA in a permuted order (the same permutation on both operands), chosen so that
// each lane's 16-byte load plus one exchange with lane^2 yields its B fragments.
//
// Lane l = 4*g + c.  After score16(): lane (g, c) holds, for query slot g (s_lo) and g + 8
// (s_hi), the UNSCALED scores of keys 4c .. 4c+3 of the group.
struct QFrag {
  uint32_t a0, a1, a2, a3;
};

// Offset (in elements) of the four physical index dimensions lane c feeds to the MMA.
__device__ __forceinline__ int qfrag_dim_offset(int lane) {
  const int c = lane & 3;
  return 8 * (c & 1) + 4 * (c >> 1);
}

// qt_row: projected queries of one row, [n_ret][16] bf16.  heads: list of retrieval-head indices
// that occupy MMA rows 0..n-1.
__device__ __forceinline__ QFrag load_qfrag(const __nv_bfloat16* qt_row, const uint8_t* heads, int n,
                                            int lane) {
  QFrag f = {0u, 0u, 0u, 0u};
  const int g = lane >> 2;
  const int off = qfrag_dim_offset(lane);
  if (g < n) {
    const uint2 v = *reinterpret_cast<const uint2*>(qt_row + (int)heads[g] * kIndexDim + off);
    f.a0 = v.x;
    f.a2 = v.y;
  }
  if (g + 8 < n) {
    const uint2 v = *reinterpret_cast<const uint2*>(qt_row + (int)heads[g + 8] * kIndexDim + off);
    f.a1 = v.x;
    f.a3 = v.y;
  }
  return f;
}

// v = this lane's 16 bytes of the 512-byte group (lane l holds bytes [16 l, 16 l + 16)).
__device__ __forceinline__ void score16(const QFrag& q, const uint4& v, int lane, float (&s_lo)[4],
                                        float (&s_hi)[4]) {
  const bool u = (lane & 2) != 0;  // lanes with u == 0 loaded an even key, u == 1 an odd key
  const uint32_t send0 = u ? v.x : v.z;
  const uint32_t send1 = u ? v.y : v.w;
  const uint32_t r0 = __shfl_xor_sync(0xffffffffu, send0, 2);
  const uint32_t r1 = __shfl_xor_sync(0xffffffffu, send1, 2);
  const uint32_t e0 = u ? r0 : v.x, e1 = u ? r1 : v.y;  // even keys (tile 0)
  const uint32_t o0 = u ? v.z : r0, o1 = u ? v.w : r1;  // odd keys (tile 1)
  const float zero[4] = {0.f, 0.f, 0.f, 0.f};
  float t0[4], t1[4];
  mma_bf16_16816(t0, q.a0, q.a1, q.a2, q.a3, e0, e1, zero);
  mma_bf16_16816(t1, q.a0, q.a1, q.a2, q.a3, o0, o1, zero);
  s_lo[0] = t0[0]; s_lo[1] = t1[0]; s_lo[2] = t0[1]; s_lo[3] = t1[1];
  s_hi[0] = t0[2]; s_hi[1] = t1[2]; s_hi[2] = t0[3]; s_hi[3] = t1[3];
}

// ---- the same core on 8-bit (E4M3) index keys ----
// A 16-key group is 256 contiguous bytes, one 8-byte load per lane (lane l holds bytes [8 l, 8 l + 8): eight
// dimensions of key l / 2).  The codes are widened to fp16 (exact) and the MMA runs on fp16 operands; the projected
// queries are converted bf16 -> fp16 once (exact for magnitudes in [2^-14, 65504]).  The output layout is score16()'s.
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1, const float (&c)[4]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%10,%11,%12,%13};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t b, bool& overflow) {
  const float lo = __uint_as_float(b << 16), hi = __uint_as_float(b & 0xffff0000u);
  overflow = overflow || !(fabsf(lo) <= 65504.0f) || !(fabsf(hi) <= 65504.0f);
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// Returns false when a projected query does not fit fp16 (the caller reports RTP_ERR_UNSUPPORTED).
__device__ __forceinline__ bool qfrag_to_f16(QFrag& f) {
  bool overflow = false;
  f.a0 = bf16x2_to_f16x2(f.a0, overflow);
  f.a1 = bf16x2_to_f16x2(f.a1, overflow);
  f.a2 = bf16x2_to_f16x2(f.a2, overflow);
  f.a3 = bf16x2_to_f16x2(f.a3, overflow);
  return !overflow;
}
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes) {
  uint32_t r;
  asm("{ .reg .b16 t; cvt.u16.u32 t, %1; cvt.rn.f16x2.e4m3x2 %0, t; }" : "=r"(r) : "r"(two_codes));
  return r;
}
__device__ __forceinline__ void score16_f8(const QFrag& q, const uint2& raw, int lane, float (&s_lo)[4],
                                           float (&s_hi)[4]) {
  uint4 v;   // the lane's eight dimensions as fp16, in the order score16() expects them
  v.x = e4m3x2_to_f16x2(raw.x);
  v.y = e4m3x2_to_f16x2(raw.x >> 16);
  v.z = e4m3x2_to_f16x2(raw.y);
  v.w = e4m3x2_to_f16x2(raw.y >> 16);
  const bool u = (lane & 2) != 0;
  const uint32_t send0 = u ? v.x : v.z;
  const uint32_t send1 = u ? v.y : v.w;
  const uint32_t r0 = __shfl_xor_sync(0xffffffffu, send0, 2);
  const uint32_t r1 = __shfl_xor_sync(0xffffffffu, send1, 2);
  const uint32_t e0 = u ? r0 : v.x, e1 = u ? r1 : v.y;
  const uint32_t o0 = u ? v.z : r0, o1 = u ? v.w : r1;
  const float zero[4] = {0.f, 0.f, 0.f, 0.f};
  float t0[4], t1[4];
  mma_f16_16816(t0, q.a0, q.a1, q.a2, q.a3, e0, e1, zero);
  mma_f16_16816(t1, q.a0, q.a1, q.a2, q.a3, o0, o1, zero);
  s_lo[0] = t0[0]; s_lo[1] = t1[0]; s_lo[2] = t0[1]; s_lo[3] = t1[1];
  s_hi[0] = t0[2]; s_hi[1] = t1[2]; s_hi[2] = t0[3]; s_hi[3] = t1[3];
}

// Final score value: temperature applied in fp32, -0 folded into +0 so that equal scores have
// equal ordered keys.
__device__ __forceinline__ float finish_score(float raw, float scale) {
  return __fadd_rn(__fmul_rn(raw, scale), 0.0f);
}

// Closed interval [raw_lo, raw_hi] of unscaled MMA outputs whose finished score has an ordered key in
// [key_lo, key_hi] (finish_score is monotone, so the preimage of a key interval is an interval; it is
// empty, raw_lo > raw_hi, when no float maps into it).  64 bisection steps.
__device__ __forceinline__ void raw_preimage(float scale, uint32_t key_lo, uint32_t key_hi, float& raw_lo, float& raw_hi) {
  const uint32_t kmin = okey(-3.4028234e38f), kmax = okey(3.4028234e38f);
  // smallest raw key with key(finish) >= key_lo
  uint32_t a = kmin, b = kmax;   // answer in [a, b]; if even kmax fails the interval is empty
  if (okey(finish_score(okey_to_float(a), scale)) >= key_lo) b = a;
  while (a + 1 < b) {
    const uint32_t mid = a + ((b - a) >> 1);
    if (okey(finish_score(okey_to_float(mid), scale)) >= key_lo) b = mid; else a = mid;
  }
  raw_lo = okey_to_float(b);
  // largest raw key with key(finish) <= key_hi
  a = kmin; b = kmax;
  if (okey(finish_score(okey_to_float(b), scale)) <= key_hi) a = b;
  while (a + 1 < b) {
    const uint32_t mid = a + ((b - a) >> 1);
    if (okey(finish_score(okey_to_float(mid), scale)) <= key_hi) a = mid; else b = mid;
  }
  raw_hi = okey_to_float(a);
}

// Warp-cooperative search on the ordered keys a <= k <= b for the smallest k with pred(k), pred monotone (false ..
// true).  Returns b + 1 (as a 64-bit value) when pred(b) is false.  Every lane probes one point per step, so a 32-bit
// range needs seven steps.  All 32 lanes must call it with the same arguments.
template <class Pred>
__device__ __forceinline__ unsigned long long warp_search_first(uint32_t a, uint32_t b, int lane, Pred pred) {
  if (!pred(b)) return (unsigned long long)b + 1ull;
  while (a < b) {   // the answer lies in [a, b]
    const unsigned long long w = (unsigned long long)(b - a);
    const uint32_t p = a + (uint32_t)((w * (unsigned long long)(lane + 1)) / 33ull);   // in [a, b)
    const uint32_t m = __ballot_sync(0xffffffffu, pred(p));
    const int f = m ? __ffs(m) - 1 : 32;                                                // first lane whose probe holds
    const uint32_t p_f = __shfl_sync(0xffffffffu, p, f & 31), p_before = __shfl_sync(0xffffffffu, p, (f + 31) & 31);
    if (f < 32) b = p_f;
    if (f > 0) a = p_before + 1u;
  }
  return a;
}


// Physical page of a block-table entry.  An entry outside [0, num_pages) (a corrupt table) is read as page 0, so that
// no kernel leaves the caches; kernels that have a status word also record RTP_ERR_INVALID for it.
// Kernels of the decode chain are launched with programmatic stream serialization: a kernel may be set up and start
// while its predecessor in the stream is still running, and waits here (first statement, before any exit) until that
// predecessor has completed and its writes are visible.  Every kernel of the chain waits, so completion is transitive.
// A no-op for a kernel launched the ordinary way.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Block-table entry (within a sequence's row) of logical page `page` of this view's pool.
__device__ __forceinline__ int page_entry(const CacheView& cv, int page) {
  return (cv.ring_pages > 0 && page >= cv.sink_pages) ? cv.sink_pages + (page - cv.sink_pages) % cv.ring_pages : page;
}
__device__ __forceinline__ int safe_phys(const CacheView& cv, int64_t entry, int32_t* status = nullptr) {
  const int phys = __ldg(cv.block_table + entry);
  if ((unsigned)phys < (unsigned)cv.num_pages) return phys;
  set_status(status, RTP_ERR_INVALID);
  return 0;
}

// Address of the 2 KB index-key slice of (logical page, index head) of a sequence.
__device__ __forceinline__ const __nv_bfloat16* ikey_page_ptr(const CacheView& cv, int seq, int page,
                                                               int ih) {
  const int phys = safe_phys(cv, (int64_t)seq * cv.max_pages + page);
  return cv.ikey + ((int64_t)phys * cv.n_ih + ih) * (kPage * kIndexDim);
}

// The same for an 8-bit index-key cache (1 KB per page and index head).
__device__ __forceinline__ const uint8_t* ikey_page_ptr8(const CacheView& cv, int seq, int page, int ih) {
  const int phys = safe_phys(cv, (int64_t)seq * cv.max_pages + page);
  return reinterpret_cast<const uint8_t*>(cv.ikey) + ((int64_t)phys * cv.n_ih + ih) * (kPage * kIndexDim);
}

// 2^x on the special-function unit (about 2 ulp; inputs of -inf give 0).
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

}  // namespace rtp
