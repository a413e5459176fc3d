// Softmax-mass histograms shared by the two top-p selection kernels (Eq. 5): level-1 binning of M - s, fixed-point
// mass accumulators with native 32-bit shared-memory adds, and the arithmetic that turns a chosen level-1 bin into
// an exact interval of ordered score keys.
#pragma once

#include "rtp_device.cuh"

namespace rtp {

constexpr int kBins = 64;                 // bins per level
constexpr float kL1Scale = 2.0f;          // level-1 bins per unit of d = M - s
constexpr float kLog2eH = 1.4426950408889634f;
// A key adds q = round(e_rel * 2^20) to its bin with one native 32-bit shared-memory add; the returned old value
// tells whether the sum wrapped, and then (rarely) a second add counts the carry in the next word.  e_rel = mass
// relative to the bin's (level 1) or the bucket's (key levels) upper end, in (e^-0.5, 1]: every key adds at
// least kMinQ, which bounds the number of keys of a bin by its sum.
constexpr float kMinQ = 634880.0f;        // (floor(e^-0.5 * 1024) - 1) * 1024

// Level-1 bin of a score.  M is an INTEGER not below any score of the row (the row maximum rounded up), so the bins
// lie on a grid that does not depend on M: with g(s) = the integer nearest to -2 s (ties to even), the bin is
// 2 M + g(s), clamped to 63; bin b holds M - s in [b/2 - 1/4, b/2 + 1/4] and the last bin pools everything below.
// Two histograms of the same row taken against different integers M, M' therefore differ by a shift of 2 (M' - M)
// bins exactly, whatever the rounding of s: partial histograms can be taken before the row maximum is known.
// Adding 1.5 * 2^23 leaves g(s) in the low mantissa bits, so no float <-> int conversion instruction is needed; the
// same arithmetic serves the histogram pass and the search that turns a bin into a key interval.
constexpr float kMagic = 12582912.0f;     // 1.5 * 2^23
constexpr float kL1MaxAbs = 262144.0f;    // |M| must stay below 2^18: then every step below is exact
// g(s) (scores far below any supported M are clamped first: they fall into the pooled bin either way)
__device__ __forceinline__ float l1_grid(float s) { return fmaf(fmaxf(s, -4.0f * kL1MaxAbs), -kL1Scale, kMagic) - kMagic; }
__device__ __forceinline__ int l1_bin_f(float M, float s, float& bin_f) {
  const float t = fminf(fmaf(kL1Scale, M, l1_grid(s)), (float)(kBins - 1)) + kMagic;
  bin_f = t - kMagic;
  return __float_as_int(t) & (kBins - 1);
}
// The integer reference of a row whose largest score is m (kept inside the range in which l1_bin_f is exact; a row
// beyond it is refused when it is resolved).
__device__ __forceinline__ float l1_anchor(float m) {
  return fminf(fmaxf(ceilf(m), -2.0f * kL1MaxAbs), 2.0f * kL1MaxAbs) + 0.0f;
}

__device__ __forceinline__ int l1_bin(float M, float s) {
  float f;
  return l1_bin_f(M, s, f);
}
// log2 of the level-1 contribution of a score, 2^20 = the bin's upper end: exp(-((M - s) - (bin/2 - 1/4))) * 2^20
__device__ __forceinline__ float l1_mass_arg(float M, float s, float bin_f) {
  return fmaf(bin_f, 0.5f * kLog2eH, fmaf(M - s, -kLog2eH, 20.0f - 0.25f * kLog2eH));
}
// factor that turns the accumulated sum of level-1 bin b into mass relative to exp(M)
__device__ __forceinline__ float l1_bin_scale(int b) {
  return fast_ex2(-kLog2eH * (0.5f * (float)b - 0.25f) - 20.0f);
}
// upper / lower end of level-1 bin b as scores
__device__ __forceinline__ float l1_bin_hi(float M, int b) { return M - ((float)b - 0.5f) / kL1Scale; }
__device__ __forceinline__ float l1_bin_lo(float M, int b) { return M - ((float)b + 0.5f) / kL1Scale; }

// Adds round(2^x) (x <= 20) to an accumulator {sum mod 2^32, carries} in shared memory.
__device__ __forceinline__ void add_mass(uint32_t* acc, float x) {
  // nearest integer to 2^x through the mantissa of (2^x + 2^23): no conversion instruction
  // (x can exceed 20 by a rounding error: a contribution a few units above 2^20 is as good as any)
  const uint32_t q = __float_as_uint(fast_ex2(x) + 8388608.0f) - 0x4b000000u;
  const uint32_t old = atomicAdd(acc, q);
  if (old + q < old) atomicAdd(acc + 1, 1u);
}
// The same contribution at 2^17 (x is still the 2^20-scale logarithm), added with a reduction that returns nothing:
// the thread does not wait for it.  The caller bounds the number of adds per bin so that the 32-bit sum cannot wrap.
__device__ __forceinline__ void add_mass17(uint32_t* acc, float x) {
  const uint32_t q = __float_as_uint(fast_ex2(x - 3.0f) + 8388608.0f) - 0x4b000000u;
  asm volatile("red.shared.add.u32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(acc)), "r"(q) : "memory");
}
__device__ __forceinline__ float acc_mass(uint32_t sum, uint32_t carries) {   // in units of 2^-20
  return (float)carries * 4294967296.0f + (float)sum;
}

// Exact interval [klo, khi] of ordered keys whose level-1 bin is `bin` (for a row maximum M): l1_bin is monotone in
// the key, so both ends are found by bisection between two keys that lie safely outside the bin.
__device__ __forceinline__ void l1_bin_keys(float M, int bin, uint32_t& klo, uint32_t& khi) {
  const float hi_s = l1_bin_hi(M, bin), lo_s = l1_bin_lo(M, bin);
  const float pad = 1e-5f * fmaxf(1.0f, fmaxf(fabsf(hi_s), fabsf(lo_s))) + 1e-3f;
  const uint32_t lo = okey(finish_score(lo_s - pad, 1.0f));
  const uint32_t hi = okey(finish_score(fminf(hi_s + pad, M), 1.0f));
  uint32_t a = lo, b = hi;              // klo = smallest key with bin <= `bin`
  if (l1_bin(M, okey_to_float(a)) <= bin) b = a;
  while (a + 1 < b) {
    const uint32_t mid = a + ((b - a) >> 1);
    if (l1_bin(M, okey_to_float(mid)) <= bin) b = mid; else a = mid;
  }
  klo = b;
  a = klo; b = hi;                      // khi = largest key with bin >= `bin`
  if (l1_bin(M, okey_to_float(b)) >= bin) a = b;
  while (a + 1 < b) {
    const uint32_t mid = a + ((b - a) >> 1);
    if (l1_bin(M, okey_to_float(mid)) >= bin) a = mid; else b = mid;
  }
  khi = a;
}

// l1_bin_keys() with the work spread over a warp (same result).
__device__ __forceinline__ void l1_bin_keys_warp(float M, int bin, int lane, uint32_t& klo, uint32_t& khi) {
  const float hi_s = l1_bin_hi(M, bin), lo_s = l1_bin_lo(M, bin);
  const float pad = 1e-5f * fmaxf(1.0f, fmaxf(fabsf(hi_s), fabsf(lo_s))) + 1e-3f;
  const uint32_t lo = okey(finish_score(lo_s - pad, 1.0f));
  const uint32_t hi = okey(finish_score(fminf(hi_s + pad, M), 1.0f));
  // bins decrease with the key: klo = first key with bin <= `bin`, khi = the key before the first with bin < `bin`
  klo = (uint32_t)warp_search_first(lo, hi, lane, [&](uint32_t k) { return l1_bin(M, okey_to_float(k)) <= bin; });
  khi = (uint32_t)(warp_search_first(lo, hi, lane, [&](uint32_t k) { return l1_bin(M, okey_to_float(k)) < bin; }) - 1ull);
}

}  // namespace rtp
