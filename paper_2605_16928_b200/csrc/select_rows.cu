// S2-S4 for explicit rows (the decode path): fused indexer scan + top-p selection (Eq. 5).
//
// The context of one (row, index head) unit is split over many CTAs.  The index keys are read once:
//   scores       every key is scored (MMA, see score16) for the unit's heads; the fp32 scores are stored, 4 bytes per
//                (head, key), and the row maxima M are taken (atomicMax on the ordered key).
// The other passes read the stored scores (half the bytes of the keys for four heads, no MMA, and at the usual sizes
// still in the L2 cache):
//   level 1      64-bin histogram of softmax mass over d = M - s in steps of 1/2, fixed point, one native
//                shared-memory add per score, merged into global memory; the unit's last CTA to finish (ticket
//                counter, nobody waits) finds Z and the bin in which the cumulative mass reaches p * Z and turns
//                it into an exact interval of ordered keys;
//   key levels   six more key bits per pass inside that interval, with exact counts, until the bucket holds at most
//                kCandCap keys (or a single key value);
//   compaction   every key above the bucket is counted and emitted, keys inside it become candidates;
//   finalize     one CTA per (row, head) sorts the candidates by (score desc, position asc) and takes the shortest
//                prefix that reaches the target mass.
#include "mass_hist.cuh"
#include "row_scan.cuh"

namespace rtp {

namespace {

using namespace rowscan;
constexpr int kHeadsPerCta = 4;

__global__ void sel_init_kernel(const CacheView cv, const Dims d, const Rows rows, SelState* state,
                                int64_t n_rowheads, uint32_t* zero_words, int64_t n_zero_words) {
  chain_wait();
  const int64_t i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  // merged histograms, counts and tickets start at zero (this replaces a separate memset)
  for (int64_t i = i0; i < n_zero_words; i += stride) zero_words[i] = 0u;
  for (int64_t i = i0; i < n_rowheads; i += stride) {
    const int64_t r = i / d.n_ret;
    const int seq = rows.row_seq(r);
    int n_keys = rows.row_pos(r) + 1;
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;   // (never beyond the block table)
    n_keys = max(0, min(n_keys, sl));
    SelState s = {};
    s.n_keys = n_keys;
    const bool every = d.top_k > 0 ? d.top_k >= n_keys : d.top_p >= 1.0f;
    s.mode = (every || n_keys <= 1) ? kSelectAll : kRefine;
    s.hi_key = 0xffffffffu;
    state[i] = s;
  }
}

// The last CTA of a (row, index head) unit to finish a pass resolves it: every CTA publishes its partial results,
// fences, and takes a ticket; the one that draws the last ticket sees all of them.  Nobody waits.
__device__ __forceinline__ bool take_last_ticket(uint32_t* ticket, uint32_t n_ctas) {
  __shared__ int s_is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t t = atomicAdd(ticket, 1u);
    s_is_last = (t == n_ctas - 1u) ? 1 : 0;
    if (s_is_last) *ticket = 0u;   // ready for the next pass
  }
  __syncthreads();
  if (s_is_last) __threadfence();
  return s_is_last != 0;
}

// ---- pass 1: scores of the unit's keys, written once for the later passes, and the row maximum -----------------------
// scores: float [rows * retrieval heads][l_pad]; entry n of a row holds finish_score(q~ . k~_n) for n < n_keys.
template <bool NH4, bool F8>
__global__ void __launch_bounds__(kThreads) sel_score_kernel(const CacheView cv, const Dims d, const HeadMaps hm,
                                                             const Rows rows, const __nv_bfloat16* __restrict__ qt,
                                                             SelState* __restrict__ state, float* __restrict__ scores,
                                                             const int64_t l_pad, int n_splits, int32_t* status) {
  chain_wait();
  __shared__ float s_max[kWarps][16];
  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, status);
  if (x.p_lo >= x.p_hi) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  QFrag qf = load_qfrag(qt + x.r * d.n_ret * kIndexDim, hm.ih_heads[x.ih], x.nh, lane);
  if (F8 && !qfrag_to_f16(qf)) set_status(status, RTP_ERR_UNSUPPORTED);   // a projected query beyond fp16's range
  const int slot_a = elem_slot<NH4>(lane, 0), slot_b = NH4 ? slot_a : elem_slot<NH4>(lane, 4);
  float* row_a = slot_a < x.nh ? scores + (x.r * d.n_ret + hm.ih_heads[x.ih][slot_a]) * l_pad : nullptr;
  float* row_b = (!NH4 && slot_b < x.nh) ? scores + (x.r * d.n_ret + hm.ih_heads[x.ih][slot_b]) * l_pad : nullptr;
  float mx_a = -INFINITY, mx_b = -INFINITY;
  uint4 v[4], vn[4];
  if (x.p_lo + warp < x.p_hi) load_page<F8>(cv, x, x.p_lo + warp, lane, vn);
  for (int p = x.p_lo + warp; p < x.p_hi; p += kWarps) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = vn[i];
    if (p + kWarps < x.p_hi) load_page<F8>(cv, x, p + kWarps, lane, vn);   // in flight while this page is worked on
    const bool tail = (p + 1) * kPage > x.n_keys;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s_lo[4], s_hi[4];
      if (F8) score16_f8(qf, make_uint2(v[i].x, v[i].y), lane, s_lo, s_hi); else score16(qf, v[i], lane, s_lo, s_hi);
      const LaneElems<NH4> el = lane_elems<NH4>(s_lo, s_hi, lane);
      const int n0 = p * kPage + i * 16 + el.koff[0];
      // (a page lies inside l_pad whatever n_keys is: entries beyond the row's keys are written and never read)
      if (NH4) {
        if (row_a)
          *reinterpret_cast<float2*>(row_a + n0) =
              make_float2(finish_score(el.raw[0], d.score_scale), finish_score(el.raw[1], d.score_scale));
      } else {
        if (row_a)
          *reinterpret_cast<float4*>(row_a + n0) =
              make_float4(finish_score(el.raw[0], d.score_scale), finish_score(el.raw[1], d.score_scale),
                          finish_score(el.raw[2], d.score_scale), finish_score(el.raw[3], d.score_scale));
        if (row_b)
          *reinterpret_cast<float4*>(row_b + n0) =
              make_float4(finish_score(el.raw[4], d.score_scale), finish_score(el.raw[5], d.score_scale),
                          finish_score(el.raw[6], d.score_scale), finish_score(el.raw[7], d.score_scale));
      }
#pragma unroll
      for (int e = 0; e < LaneElems<NH4>::kN; ++e) {
        if (tail && p * kPage + i * 16 + el.koff[e] >= x.n_keys) continue;
        if (NH4 || e < 4) mx_a = fmaxf(mx_a, el.raw[e]); else mx_b = fmaxf(mx_b, el.raw[e]);
      }
    }
  }
  mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
  mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
  if (NH4) mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 16));
  mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
  mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
  if ((lane & 3) == 0) {
    const int g = lane >> 2;
    if (NH4) {
      if (g < 4) s_max[warp][g] = mx_a;
    } else {
      s_max[warp][g] = mx_a;
      s_max[warp][g + 8] = mx_b;
    }
  }
  __syncthreads();
  if (threadIdx.x < x.nh) {
    float m = -INFINITY;
    for (int w = 0; w < kWarps; ++w) m = fmaxf(m, s_max[w][threadIdx.x]);
    // the maximum was taken on unscaled MMA outputs; scaling by a positive factor is monotone.  What the later passes
    // need is a reference not below any score, an integer (see l1_bin_f): the maximum rounded up
    if (m > -INFINITY) atomicMax(&state[x.r * d.n_ret + hm.ih_heads[x.ih][threadIdx.x]].max_key, okey(l1_anchor(finish_score(m, d.score_scale))));
  }
}

// The later passes read the stored scores: the CTA's share of a row is keys [k_lo, k_hi), four consecutive keys per
// thread and step (one 16-byte load).
constexpr int kLoads = 4;   // 16-byte loads a thread keeps in flight in the passes over the stored scores
struct KeySpan {
  int k_lo, k_hi;
};
__device__ __forceinline__ KeySpan key_span(const RowCtx& x) {
  KeySpan s;
  s.k_lo = x.p_lo * kPage;
  s.k_hi = min(x.p_hi * kPage, x.n_keys);
  return s;
}
__device__ __forceinline__ float4 ld_scores4(const float* p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

constexpr float kCountScale = 9.5367431640625e-07f;   // 2^-20: a key of the fixed-budget selector adds 2^20 to its bin

// Level-1 resolve by one warp: lane l holds the sums of bins 2l and 2l + 1 (bin 0 is the top) as q0, q1 (2^20 fixed
// point relative to the bin's upper end) and whether the bins are populated.  Finds Z and the bin in which the cumulative
// mass reaches the target and turns it into an exact interval of ordered keys in *st.
__device__ __forceinline__ void l1_resolve_warp(const Dims& d, const float M, const float q0, const float q1,
                                                const bool has0, const bool has1, const int lane, const int list_cap,
                                                SelState* st, int32_t* status) {
  const bool by_count = d.top_k > 0;
  if (!(fabsf(M) < kL1MaxAbs)) {   // scores beyond the supported range (or not finite): every key is kept
    if (lane == 0) {
      st->mode = kSelectAll;
      set_status(status, RTP_ERR_UNSUPPORTED);
    }
    return;
  }
  const int b0 = 2 * lane, b1 = 2 * lane + 1;
  const float m0 = q0 * (by_count ? kCountScale : l1_bin_scale(b0)), m1 = q1 * (by_count ? kCountScale : l1_bin_scale(b1));
  float inc = m0 + m1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  const float Z = __shfl_sync(0xffffffffu, inc, 31);
  // (counts are small integers: their sums are exact and the target needs no margin)
  const float target = by_count ? (float)d.top_k : d.top_p * Z * (1.0f + kMassMargin);
  const float run = inc - (m0 + m1);
  int found = 64, last = -1;
  if (has0) {
    last = b0;
    if (run + m0 >= target) found = b0;
  }
  if (has1) {
    last = b1;
    if (found == 64 && run + m0 + m1 >= target) found = b1;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
    last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
  }
  if (found == 64) found = last;   // rounding left the target just out of reach: lowest populated bin
  if (found < 0) {
    if (lane == 0) {               // empty histogram: cannot happen for a non-empty row
      st->mode = kSelectAll;
      set_status(status, RTP_ERR_UNSUPPORTED);
    }
    return;
  }
  {
    // the lane that owns the bin hands its figures to the warp; the interval searches are warp-wide
    const int owner = found >> 1;
    const bool first = (found & 1) == 0;
    const float above = __shfl_sync(0xffffffffu, first ? run : run + m0, owner);
    const float q = __shfl_sync(0xffffffffu, first ? q0 : q1, owner);
    uint32_t klo = 0u, khi = 0u;
    // Top-P: a cut inside the pooled last bin (mass below 1e-13 per key) keeps every key.  The fixed budget counts
    // keys, so its cut can fall there: the bucket is then every key from the bottom up to the pool's upper end.
    const bool pooled = found == kBins - 1 && !by_count;
    if (!pooled) {
      l1_bin_keys_warp(M, found, lane, klo, khi);
      if (found == kBins - 1) klo = 0u;
    }
    if (lane == 0) {
      st->M = M;
      st->Z = Z;
      st->target = target;
      st->mass_above = above;
      if (pooled) {
        st->mode = kSelectAll;       // the cut falls into the pooled tail: take every key
      } else {
        const uint32_t span = khi - klo + 1u;
        const int bits = span > 1u ? 32 - __clz(span - 1u) : 0;
        st->lo_key = klo;
        st->hi_key = khi;
        st->span = span;
        st->shift = max(0, bits - 6);
        st->ref_s = l1_bin_hi(M, found);
        st->e_ref = by_count ? 1.0f : fast_ex2(-kLog2eH * (0.5f * (float)found - 0.25f));
        if (q < 0.999f * kMinQ * (float)list_cap) st->mode = kCollect;   // fewer than list_cap keys in the bin
      }
    }
  }
}

// ---- pass 2: level-1 mass histogram over M - s, resolved by the unit's last CTA ----------------------------------
__global__ void __launch_bounds__(kThreads) sel_l1_kernel(const CacheView cv, const Dims d, const HeadMaps hm,
                                                          const Rows rows, const float* __restrict__ scores,
                                                          const int64_t l_pad, SelState* __restrict__ state,
                                                          unsigned long long* __restrict__ g_mass,
                                                          uint32_t* __restrict__ tickets, int n_splits, const int list_cap,
                                                          int32_t* status) {
  chain_wait();
  // One private histogram per warp and head of the chunk, 2^17 fixed point, added to with reductions that return
  // nothing (the thread does not wait for them): a warp sees at most 16384 keys per head between two merges
  // (select_splits) and a key adds at most 2^17 (+ rounding), so a 32-bit sum cannot wrap.
  __shared__ uint32_t hist[kHeadsPerCta][kWarps][kBins];
  __shared__ float s_M[16];
  __shared__ int s_on[16];
  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, nullptr);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x < 16) {
    int on = 0;
    float M = 0.f;
    if (threadIdx.x < x.nh) {
      const SelState* st = state + (x.r * d.n_ret + hm.ih_heads[x.ih][threadIdx.x]);
      on = st->mode == kRefine && st->n_keys > 0;
      M = okey_to_float(st->max_key);
    }
    s_on[threadIdx.x] = on;
    s_M[threadIdx.x] = M;
  }
  for (int i = threadIdx.x; i < kHeadsPerCta * kWarps * kBins; i += kThreads) (&hist[0][0][0])[i] = 0u;
  __syncthreads();
  int any = 0;
  for (int j = 0; j < x.nh; ++j) any |= s_on[j];
  if (!any) return;   // the same decision in every CTA of the unit

  const KeySpan ks = key_span(x);
  const bool by_count = d.top_k > 0;   // fixed budget: every key weighs the same, the "mass" is a count
  for (int j0 = 0; j0 < x.nh; j0 += kHeadsPerCta) {   // four heads at a time: their loads are in flight together
    const float* row[kHeadsPerCta];
    float Mj[kHeadsPerCta];
    bool on[kHeadsPerCta];
#pragma unroll
    for (int jj = 0; jj < kHeadsPerCta; ++jj) {
      on[jj] = j0 + jj < x.nh && s_on[j0 + jj];
      row[jj] = scores + (x.r * d.n_ret + (on[jj] ? hm.ih_heads[x.ih][j0 + jj] : 0)) * l_pad;
      Mj[jj] = on[jj] ? s_M[j0 + jj] : 0.f;
    }
    for (int n0 = ks.k_lo + 4 * (int)threadIdx.x; n0 < ks.k_hi; n0 += 4 * kThreads) {
      float4 v[kHeadsPerCta];
#pragma unroll
      for (int jj = 0; jj < kHeadsPerCta; ++jj) v[jj] = on[jj] ? ld_scores4(row[jj] + n0) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int jj = 0; jj < kHeadsPerCta; ++jj) {
        if (!on[jj]) continue;   // uniform
        const float s4[4] = {v[jj].x, v[jj].y, v[jj].z, v[jj].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (n0 + e >= ks.k_hi) continue;
          float bin_f;
          const int bin = l1_bin_f(Mj[jj], s4[e], bin_f);
          const float arg = l1_mass_arg(Mj[jj], s4[e], bin_f);
          add_mass17(&hist[jj][warp][bin], by_count ? 20.0f : arg);
        }
      }
    }
    __syncthreads();
    {
      const int jj = threadIdx.x / kBins, bin = threadIdx.x % kBins;   // 256 threads = 4 heads x 64 bins
      unsigned long long tot = 0ull;
      for (int w = 0; w < kWarps; ++w) {
        tot += (unsigned long long)hist[jj][w][bin] << 3;   // back to the 2^20 scale of the merged histogram
        hist[jj][w][bin] = 0u;
      }
      if (tot) atomicAdd(g_mass + (x.r * d.n_ret + hm.ih_heads[x.ih][j0 + jj]) * kBins + bin, tot);
    }
    __syncthreads();
  }
  if (!take_last_ticket(tickets + blockIdx.x, gridDim.y)) return;

  // ---- resolve: one warp per head; lane l looks at bins 2l, 2l+1 (bin 0 is the top) ----
  for (int j = warp; j < x.nh; j += kWarps) {
    if (!s_on[j]) continue;
    const int64_t rh = x.r * d.n_ret + hm.ih_heads[x.ih][j];
    unsigned long long* gm = g_mass + rh * kBins;
    const int b0 = 2 * lane, b1 = 2 * lane + 1;
    const unsigned long long u0 = __ldcg(gm + b0), u1 = __ldcg(gm + b1);
    gm[b0] = 0ull;
    gm[b1] = 0ull;
    l1_resolve_warp(d, s_M[j], __ull2float_rn(u0), __ull2float_rn(u1), u0 != 0ull, u1 != 0ull, lane, list_cap, state + rh, status);
  }
}

// Key-level resolve by one warp: lane l holds the sums (2^20 fixed point relative to the bucket's reference) and the
// key counts of bins 63 - 2l and 62 - 2l (bin 63 is the top) of the bucket's current six key bits.  Narrows the bucket in
// *st to the bin in which the cumulative mass reaches the target.
__device__ __forceinline__ void key_resolve_warp(const Dims& d, const float q0, const float q1, const uint32_t c0,
                                                 const uint32_t c1, const int lane, const int list_cap, SelState* st,
                                                 int32_t* status) {
  const float sc = st->e_ref * 9.5367431640625e-07f;   // 2^-20
  const float m0 = q0 * sc, m1 = q1 * sc;
  float inc = m0 + m1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  const float above0 = st->mass_above, target = st->target;
  const float run = above0 + inc - (m0 + m1);
  int found = 64, last = -1;   // order index from the top
  if (c0) {
    last = 2 * lane;
    if (run + m0 >= target) found = 2 * lane;
  }
  if (c1) {
    last = 2 * lane + 1;
    if (found == 64 && run + m0 + m1 >= target) found = 2 * lane + 1;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
    last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
  }
  if (found == 64) found = last;
  __syncwarp();
  if (found < 0) {
    if (lane == 0) {               // a chosen bucket always holds a key
      st->mode = kSelectAll;
      set_status(status, RTP_ERR_UNSUPPORTED);
    }
    return;
  }
  {
    const int owner = found >> 1;
    const bool first = (found & 1) == 0;
    const int bin = 63 - found;
    const uint32_t cnt = __shfl_sync(0xffffffffu, first ? c0 : c1, owner);
    const float above = __shfl_sync(0xffffffffu, first ? run : run + m0, owner);
    const int shift = st->shift;
    const uint32_t ofs = (uint32_t)bin << shift;
    const uint32_t lo_key = st->lo_key + ofs;
    const uint32_t sub_span = min(1u << shift, st->span - ofs);
    if (lane == 0) {
      st->mass_above = above;
      st->lo_key = lo_key;
      st->hi_key = lo_key + (sub_span - 1u);
      st->span = sub_span;
      st->bucket_cnt = (int)cnt;
      st->shift = max(0, shift - 6);
      if (cnt <= (uint32_t)list_cap)
        st->mode = kCollect;
      else if (sub_span == 1u)
        st->mode = kTieScan;         // more than list_cap equal scores straddle the cut
    }
    __syncwarp();
  }
}

// ---- pass 3 (repeated): 64-bin mass histogram of the next six key bits inside the bucket --------------------------
// Only a small share of the scores falls into a head's bucket: a warp appends those hits to a queue in shared
// memory and works them off 32 at a time, one hit per lane.
struct KeyParams {   // per head slot, shared memory
  uint32_t base_key;
  int32_t shift;
  float ref_s;
};

__global__ void __launch_bounds__(kThreads) sel_key_kernel(const CacheView cv, const Dims d, const HeadMaps hm,
                                                           const Rows rows, const float* __restrict__ scores,
                                                           const int64_t l_pad,
                                                           SelState* __restrict__ state, unsigned long long* __restrict__ g_mass,
                                                           uint32_t* __restrict__ g_cnt, uint32_t* __restrict__ tickets,
                                                           int n_splits, int max_levels, const int list_cap, int32_t* status) {
  chain_wait();
  __shared__ uint32_t hist[16][kBins][3];   // {sum, carries, count}
  __shared__ KeyParams kp[16];
  __shared__ uint32_t s_span[16];
  __shared__ int s_on[16];
  RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, nullptr);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t n_ctas = gridDim.y;
  // The first level is split over the unit's CTAs.  The CTA that resolves it goes on alone with whatever is still
  // unresolved (rare: dense clusters of nearly equal scores), scanning the whole unit, up to max_levels in all.
#pragma unroll 1
  for (int level = 0; level < max_levels; ++level) {
  if (threadIdx.x < 16) {
    int on = 0;
    uint32_t span = 0u;
    KeyParams k = {0u, 0, 0.f};
    if (threadIdx.x < x.nh) {
      const volatile SelState* st = state + (x.r * d.n_ret + hm.ih_heads[x.ih][threadIdx.x]);
      on = st->mode == kRefine && st->n_keys > 0;
      if (on) {
        span = st->span;
        k.base_key = st->lo_key;
        k.shift = st->shift;
        k.ref_s = st->ref_s;
      }
    }
    s_on[threadIdx.x] = on;
    s_span[threadIdx.x] = span;
    kp[threadIdx.x] = k;
  }
  for (int i = threadIdx.x; i < 16 * kBins * 3; i += kThreads) (&hist[0][0][0])[i] = 0u;
  __syncthreads();
  int any = 0;
  for (int j = 0; j < x.nh; ++j) any |= s_on[j];
  if (!any) return;   // the same decision in every CTA of the unit

  // hits are rare (the bucket holds a few per cent of the keys at most): each is added where it is found
  const KeySpan ks = key_span(x);
  for (int j = 0; j < x.nh; ++j) {
    if (!s_on[j]) continue;   // uniform
    const float* row = scores + (x.r * d.n_ret + hm.ih_heads[x.ih][j]) * l_pad;
    const uint32_t base_key = kp[j].base_key, span = s_span[j];
    const int shift = kp[j].shift;
    const float ref_s = kp[j].ref_s;
    const float lw = d.top_k > 0 ? 0.f : kLog2eH;   // fixed budget: every key adds 2^20
    for (int nb = ks.k_lo + 4 * (int)threadIdx.x; nb < ks.k_hi; nb += kLoads * 4 * kThreads) {
      float4 v[kLoads];
#pragma unroll
      for (int k = 0; k < kLoads; ++k) {
        const int n0 = nb + k * 4 * kThreads;
        v[k] = n0 < ks.k_hi ? ld_scores4(row + n0) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < kLoads; ++k) {
        const int n0 = nb + k * 4 * kThreads;
        const float s4[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t t = okey(s4[e]) - base_key;
          if (n0 + e < ks.k_hi && t < span) {
            uint32_t* acc = &hist[j][t >> shift][0];
            add_mass(acc, fmaf(s4[e] - ref_s, lw, 20.0f));
            atomicAdd(acc + 2, 1u);
          }
        }
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < x.nh * kBins; i += kThreads) {
    const int j = i / kBins, bin = i % kBins;
    const uint32_t n = hist[j][bin][2];
    if (n) {
      const int64_t o = (x.r * d.n_ret + hm.ih_heads[x.ih][j]) * kBins + bin;
      atomicAdd(g_mass + o, ((unsigned long long)hist[j][bin][1] << 32) | hist[j][bin][0]);
      atomicAdd(g_cnt + o, n);
    }
  }
  if (!take_last_ticket(tickets + blockIdx.x, n_ctas)) return;

  // ---- resolve: one warp per head; lane l looks at bins 63 - 2l, 62 - 2l (bin 63 is the top) ----
  for (int j = warp; j < x.nh; j += kWarps) {
    if (!s_on[j]) continue;
    const int64_t rh = x.r * d.n_ret + hm.ih_heads[x.ih][j];
    unsigned long long* gm = g_mass + rh * kBins;
    uint32_t* gc = g_cnt + rh * kBins;
    const int b0 = 63 - 2 * lane, b1 = 62 - 2 * lane;
    const unsigned long long u0 = __ldcg(gm + b0), u1 = __ldcg(gm + b1);
    const uint32_t c0 = __ldcg(gc + b0), c1 = __ldcg(gc + b1);
    gm[b0] = 0ull;
    gm[b1] = 0ull;
    gc[b0] = 0u;
    gc[b1] = 0u;
    key_resolve_warp(d, __ull2float_rn(u0), __ull2float_rn(u1), c0, c1, lane, list_cap, state + rh, status);
  }
  __threadfence();
  __syncthreads();
  x.p_lo = 0;                                   // from here on this CTA owns the whole unit
  x.p_hi = (x.n_keys + kPage - 1) >> kPageShift;
  n_ctas = 1;
  }
}

// ---- compaction -------------------------------------------------------------------------------------
// Keys above a head's bucket are counted and, when id lists are requested, emitted; keys inside it become candidates
// for the exact finish.  A CTA takes up to four heads of the unit (blockIdx.z), one after the other; a warp reads 128
// consecutive stored scores per step and ballots the hits into its two stages in shared memory, which are appended
// to the row's list / candidate array with one counter update per flush.
// The float f with  s >= f  <=>  okey(s) >= k  (or okey(s) > k with `above`) for every score s (finite or infinite, never
// NaN, never -0).  Keys at or below that of -inf give -inf (every score qualifies), keys beyond that of +inf give NaN (none).
__device__ __forceinline__ float key_floor(uint32_t k, bool above) {
  if (above) {
    if (k == 0xffffffffu) return __int_as_float(0x7fc00000);
    ++k;
  }
  if (k <= okey(-INFINITY)) return -INFINITY;
  if (k > okey(INFINITY)) return __int_as_float(0x7fc00000);
  return okey_to_float(k);   // (for k = key of +0 this is +0, for the key of -0 it is -0: both compare as zero)
}

constexpr int kIdStage = 384;     // a step adds at most 128 entries: flushed when more than 256 are staged
constexpr int kCandStageW = 256;  // flushed when more than 128 are staged

__global__ void __launch_bounds__(kThreads) sel_compact_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows, const float* __restrict__ scores,
    const int64_t l_pad, SelState* __restrict__ state, uint2* __restrict__ cand, const int list_cap,
    int32_t* __restrict__ sel_idx, int64_t sel_stride, int n_splits, int32_t* status) {
  chain_wait();
  __shared__ int id_stage[kWarps][kIdStage];
  __shared__ uint2 cand_stage[kWarps][kCandStageW];
  __shared__ int st_fill[kWarps][2];   // entries in the warp's two stages
  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, nullptr);
  const int z = blockIdx.z;
  if (z * kHeadsPerCta >= x.nh || x.p_lo >= x.p_hi) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const KeySpan ks = key_span(x);
  const bool emit_ids = sel_idx != nullptr;
  const int nj = min(kHeadsPerCta, x.nh - z * kHeadsPerCta);
#pragma unroll 1
  for (int j = 0; j < nj; ++j) {
    const int64_t rh = x.r * d.n_ret + hm.ih_heads[x.ih][z * kHeadsPerCta + j];
    SelState* st = state + rh;
    const int mode = st->mode;
    const uint32_t lo_key = st->lo_key, hi_key = st->hi_key;
    const bool all = mode == kSelectAll, bucket = mode == kCollect || mode == kTieScan, collect = mode == kCollect;
    const float* row = scores + rh * l_pad;
    // s >= f_above <=> key(s) > hi_key ("above the bucket", or every key); s >= f_lo <=> key(s) >= lo_key
    const float f_above = all ? -INFINITY : (bucket ? key_floor(hi_key, true) : __int_as_float(0x7fc00000));
    const float f_lo = collect ? key_floor(lo_key, false) : __int_as_float(0x7fc00000);
    // Hits are sparse (a few per cent of the keys): a lane that has some reserves room in its warp's stage with one
    // shared-memory add (the order inside a stage does not matter); the fills live in shared memory.
    int n_above = 0;
    if (lane == 0) {
      st_fill[warp][0] = 0;
      st_fill[warp][1] = 0;
    }
    __syncwarp();
    auto flush_ids = [&](int cnt_i) {
      int gbase = 0;
      if (lane == 0) gbase = atomicAdd(&st->emit_cnt, cnt_i);
      gbase = __shfl_sync(0xffffffffu, gbase, 0);
      for (int i = lane; i < cnt_i; i += 32)
        if (gbase + i < sel_stride) sel_idx[rh * sel_stride + gbase + i] = id_stage[warp][i];
      if (gbase + cnt_i > sel_stride && lane == 0) set_status(status, RTP_ERR_CAPACITY);
      __syncwarp();
      if (lane == 0) st_fill[warp][0] = 0;
      __syncwarp();
    };
    auto flush_cands = [&](int cnt_c) {
      int gbase = 0;
      if (lane == 0) gbase = atomicAdd(&st->cand_cnt, cnt_c);
      gbase = __shfl_sync(0xffffffffu, gbase, 0);
      for (int i = lane; i < cnt_c; i += 32)
        if (gbase + i < list_cap) cand[rh * (int64_t)list_cap + gbase + i] = cand_stage[warp][i];
      __syncwarp();
      if (lane == 0) st_fill[warp][1] = 0;
      __syncwarp();
    };
    for (int nw = ks.k_lo + 128 * warp; nw < ks.k_hi; nw += 128 * kWarps) {
      const int n0 = nw + 4 * lane;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (n0 < ks.k_hi) v = ld_scores4(row + n0);
      const float s4[4] = {v.x, v.y, v.z, v.w};
      uint32_t a_bits = 0u, c_bits = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        // float comparisons against the bucket's ends (key_floor): one instruction each instead of an ordered key
        const bool ok = n0 + e < ks.k_hi;
        const bool fa = ok && s4[e] >= f_above;
        const bool fc = ok && s4[e] >= f_lo && !(s4[e] >= f_above);
        a_bits |= (uint32_t)fa << e;
        c_bits |= (uint32_t)fc << e;
      }
      n_above += __popc(a_bits);
      if (emit_ids && a_bits) {
        int at = atomicAdd(&st_fill[warp][0], __popc(a_bits));
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((a_bits >> e) & 1u) id_stage[warp][at++] = n0 + e;
      }
      if (c_bits) {
        int at = atomicAdd(&st_fill[warp][1], __popc(c_bits));
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((c_bits >> e) & 1u) cand_stage[warp][at++] = make_uint2(okey(s4[e]), (uint32_t)(n0 + e));
      }
      __syncwarp();
      const int cnt_i = st_fill[warp][0], cnt_c = st_fill[warp][1];
      if (cnt_i > kIdStage - 128) flush_ids(cnt_i);
      if (cnt_c > kCandStageW - 128) flush_cands(cnt_c);
    }
    __syncwarp();
    if (st_fill[warp][0] > 0) flush_ids(st_fill[warp][0]);
    if (st_fill[warp][1] > 0) flush_cands(st_fill[warp][1]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n_above += __shfl_xor_sync(0xffffffffu, n_above, o);
    if (lane == 0 && n_above && !all) atomicAdd(&st->cnt_above, n_above);
  }
}

// ---- finalize ---------------------------------------------------------------------------------------
constexpr int kFinThreads = 1024;
constexpr int kFinWarps = kFinThreads / 32;
constexpr int kNoPick = 0x7fffffff;
constexpr int kFinLoads = 8;   // entries of a candidate list in global memory that a thread has in flight

// The finish of one (row, head), run by a CTA of kFinThreads threads: `row` = the row's scores (global memory, or
// shared memory in the one-kernel path for short contexts), `st` = its selection state, `gl` = its candidate list in
// global memory (ignored when `preloaded`: the st->cand_cnt <= kCandCap candidates are then in `keys` already),
// keys / keys2 = two buffers of kCandCap sort keys in shared memory.
__device__ void finalize_core(const Dims& d, const float* row, SelState* st, const uint2* gl, const int list_cap,
                              const bool preloaded, unsigned long long* keys, unsigned long long* keys2, const int64_t rh,
                              int32_t* __restrict__ sel_idx, int64_t sel_stride, int32_t* __restrict__ sel_count,
                              float* __restrict__ sel_mass, float* __restrict__ sel_thresh,
                              int32_t* __restrict__ sel_tie_last, int32_t* status) {
  __shared__ uint32_t fh[kBins][3];   // narrowing: {sum, carries, count} per bin
  __shared__ float w_sum[kFinWarps];
  __shared__ int w_cnt[kFinWarps];
  __shared__ int s_pick, s_emitted, s_last, s_bin, s_n2, s_sel;
  __shared__ float s_run, s_pick_mass, s_above;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mode = st->mode;
  const int n_keys = st->n_keys;
  int32_t* ids = sel_idx ? sel_idx + rh * sel_stride : nullptr;

  if (n_keys == 0) {
    if (tid == 0) {
      sel_count[rh] = 0;
      if (sel_mass) sel_mass[rh] = 0.f;
      if (sel_thresh) sel_thresh[rh] = 0.f;
      if (sel_tie_last) sel_tie_last[rh] = -1;
    }
    return;
  }
  if (mode == kSelectAll) {
    if (tid == 0) {
      sel_count[rh] = n_keys;
      if (sel_mass) sel_mass[rh] = 1.0f;
      if (sel_thresh) sel_thresh[rh] = -INFINITY;
      if (sel_tie_last) sel_tie_last[rh] = n_keys - 1;
      if (ids && n_keys > sel_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }
  const float M = st->M, Z = st->Z, target = st->target;
  const bool by_count = d.top_k > 0;
  float above = st->mass_above;
  int base = st->cnt_above;
  int emit_base = ids ? st->emit_cnt : base;

  bool tie = mode == kTieScan;
  uint32_t tie_key = st->lo_key;
  int tie_bucket = st->bucket_cnt;
  int n_fin = 0;   // candidates left for the exact sort

  // Forced positions (a selectable variant, off in the paper's method): the first force_sink and the newest
  // force_recent keys of the row that the regular rule (score above the threshold, or equal to it and not beyond
  // t_last) left out are appended behind the `count` regular entries.  Returns how many were added; their mass
  // (relative to exp(M), or their number under the fixed budget) is added to mass_io.  Called by every thread.
  auto add_forced = [&](uint32_t t_key, int t_last, int count, float& mass_io) -> int {
    const int n_head = min(d.force_sink, n_keys), tail_lo = max(n_head, n_keys - d.force_recent);
    const int nf = n_head + (n_keys - tail_lo);
    if (nf <= 0) return 0;   // uniform
    __syncthreads();
    if (tid == 0) s_n2 = 0;
    __syncthreads();
    float em = 0.f;
    for (int i = tid; i < nf; i += kFinThreads) {
      const int n = i < n_head ? i : tail_lo + (i - n_head);
      const float sv = row[n];   // (a generic load: the row may live in shared memory)
      const uint32_t key = okey(sv);
      if (!(key > t_key || (key == t_key && n <= t_last))) {
        const int pos = count + atomicAdd(&s_n2, 1);
        if (ids && pos < sel_stride) ids[pos] = n;
        em += by_count ? 1.0f : __expf(sv - M);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) em += __shfl_xor_sync(0xffffffffu, em, o);
    if (lane == 0) w_sum[warp] = em;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < kFinWarps; ++w) tot += w_sum[w];   // the same order in every thread and every run
    mass_io += tot;
    const int added = s_n2;
    __syncthreads();
    return added;
  };
  if (mode == kCollect) {
    // The candidates of the bucket: a list in global memory (up to list_cap entries).  A list that fits is copied to
    // shared memory at once; a longer one is narrowed where it is until the chosen part fits.
    const int n_src = min(st->cand_cnt, list_cap);
    bool in_global = !preloaded && n_src > kCandCap;
    int n = n_src;   // candidates inside [lo_key, lo_key + span)
    if (!in_global && !preloaded) {
      for (int i = tid; i < n; i += kFinThreads) {
        const uint2 cnd = gl[i];
        keys[i] = ((unsigned long long)(~cnd.x) << 32) | (unsigned long long)cnd.y;
      }
    }
    __syncthreads();
    // Narrowing: while many candidates are left, one more 64-bin mass histogram over the next six key bits of the
    // bucket on the candidate list: candidates above the chosen bin are selected (and their ids emitted), those below
    // are dropped, those inside go on.  The exact sort below then sees a short list.
    {
      uint32_t lo_key = st->lo_key, span = st->span;
      const float ref_s = st->ref_s, sc = st->e_ref * 9.5367431640625e-07f;   // 2^-20
      const float lw = by_count ? 0.f : kLog2eH;
      while ((n > 256 || in_global) && span > 1u) {
        const int bits = 32 - __clz(span - 1u);
        const int shift = max(0, bits - 6);
        for (int i = tid; i < kBins * 3; i += kFinThreads) (&fh[0][0])[i] = 0u;
        if (tid == 0) {
          s_n2 = 0;
          s_sel = 0;
        }
        __syncthreads();
        if (in_global) {
          // (the list entries of a thread are loaded several at a time: one round trip for kFinLoads of them)
          for (int i0 = tid; i0 < n_src; i0 += kFinThreads * kFinLoads) {
            uint32_t key[kFinLoads];
#pragma unroll
            for (int k = 0; k < kFinLoads; ++k) {
              const int i = i0 + k * kFinThreads;
              key[k] = i < n_src ? __ldcg(&gl[i].x) : 0u;
            }
#pragma unroll
            for (int k = 0; k < kFinLoads; ++k) {
              const uint32_t t = key[k] - lo_key;
              if (i0 + k * kFinThreads < n_src && t < span) {
                uint32_t* acc = &fh[t >> shift][0];
                add_mass(acc, fmaf(okey_to_float(key[k]) - ref_s, lw, 20.0f));
                atomicAdd(acc + 2, 1u);
              }
            }
          }
        } else {
          for (int i = tid; i < n; i += kFinThreads) {
            const uint32_t key = ~(uint32_t)(keys[i] >> 32);
            uint32_t* acc = &fh[(key - lo_key) >> shift][0];
            add_mass(acc, fmaf(okey_to_float(key) - ref_s, lw, 20.0f));
            atomicAdd(acc + 2, 1u);
          }
        }
        __syncthreads();
        if (warp == 0) {   // lane l looks at bins 63 - 2l, 62 - 2l (bin 63 is the top)
          const int b0 = 63 - 2 * lane, b1 = 62 - 2 * lane;
          const float m0 = acc_mass(fh[b0][0], fh[b0][1]) * sc, m1 = acc_mass(fh[b1][0], fh[b1][1]) * sc;
          const uint32_t c0 = fh[b0][2], c1 = fh[b1][2];
          float inc = m0 + m1;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
          }
          const float run = above + inc - (m0 + m1);
          int found = 64, last = -1;
          if (c0) {
            last = 2 * lane;
            if (run + m0 >= target) found = 2 * lane;
          }
          if (c1) {
            last = 2 * lane + 1;
            if (found == 64 && run + m0 + m1 >= target) found = 2 * lane + 1;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
            last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
          }
          if (found == 64) found = last;
          if ((found >> 1) == lane) {
            s_bin = 63 - found;
            s_above = (found & 1) ? run + m0 : run;
          }
        }
        __syncthreads();
        const int bin = s_bin;
        const int cnt_bin = (int)fh[bin][2];
        const bool to_smem = in_global && cnt_bin <= kCandCap;
        if (in_global) {
          for (int i0 = tid; i0 < n_src; i0 += kFinThreads * kFinLoads) {
            uint2 cnd[kFinLoads];
#pragma unroll
            for (int k = 0; k < kFinLoads; ++k) {
              const int i = i0 + k * kFinThreads;
              cnd[k] = i < n_src ? __ldcg(&gl[i]) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int k = 0; k < kFinLoads; ++k) {
              const uint32_t t = cnd[k].x - lo_key;
              if (i0 + k * kFinThreads < n_src && t < span) {
                const int b = (int)(t >> shift);
                if (b > bin) {
                  const int pos = atomicAdd(&s_sel, 1);
                  if (ids && emit_base + pos < sel_stride) ids[emit_base + pos] = (int)cnd[k].y;
                } else if (b == bin && to_smem) {
                  keys2[atomicAdd(&s_n2, 1)] = ((unsigned long long)(~cnd[k].x) << 32) | (unsigned long long)cnd[k].y;
                }
              }
            }
          }
        } else {
          for (int i = tid; i < n; i += kFinThreads) {
            const unsigned long long k = keys[i];
            const int b = (int)((~(uint32_t)(k >> 32) - lo_key) >> shift);
            if (b > bin) {
              const int pos = atomicAdd(&s_sel, 1);
              if (ids && emit_base + pos < sel_stride) ids[emit_base + pos] = (int)(uint32_t)k;
            } else if (b == bin) {
              keys2[atomicAdd(&s_n2, 1)] = k;
            }
          }
        }
        __syncthreads();
        above = s_above;
        base += s_sel;
        emit_base += s_sel;
        n = cnt_bin;
        const uint32_t ofs = (uint32_t)bin << shift;
        lo_key += ofs;
        span = min(1u << shift, span - ofs);
        if (!in_global || to_smem) {
          unsigned long long* t = keys;
          keys = keys2;
          keys2 = t;
          in_global = false;
        }
        __syncthreads();
      }
      if (in_global) {   // one key value with more candidates than the sort takes: exact ties
        tie = true;
        tie_key = lo_key;
        tie_bucket = n;
      }
    }
    n_fin = n;
  }
  if (mode == kCollect && !tie) {
    const int n = n_fin;
    int np = 1;
    while (np < n) np <<= 1;
    for (int i = n + tid; i < np; i += kFinThreads) keys[i] = ~0ull;
    if (tid == 0) {
      s_pick = kNoPick;
      s_run = 0.f;
      s_pick_mass = 0.f;
    }
    __syncthreads();
    // ascending order = larger score first, then smaller position.  A short list (the usual case after the narrowing) is
    // sorted by rank: every candidate counts the smaller ones (the keys are distinct: they hold the position) and goes to
    // that place of the other buffer, with one barrier; a long one (many equal scores) by a bitonic network.
    if (n <= 1024) {
      if (tid < n) {
        const unsigned long long k = keys[tid];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += keys[j] < k;
        keys2[tid < n ? rank : 0] = k;
      }
      __syncthreads();
      unsigned long long* t = keys;
      keys = keys2;
      keys2 = t;
    } else
    for (int size = 2; size <= np; size <<= 1) {
      for (int stride = size >> 1; stride > 0; stride >>= 1) {
        for (int i = tid; i < (np >> 1); i += kFinThreads) {
          const int lo = 2 * i - (i & (stride - 1));
          const int hi = lo + stride;
          const bool up = (lo & size) == 0;
          const unsigned long long a = keys[lo], b = keys[hi];
          if ((a > b) == up) {
            keys[lo] = b;
            keys[hi] = a;
          }
        }
        __syncthreads();
      }
    }
    // prefix masses in sorted order, 256 candidates per round
    for (int r0 = 0; r0 < n; r0 += kFinThreads) {
      if (s_pick != kNoPick) break;  // uniform: written before the barrier that ends each round
      const int i = r0 + tid;
      float e = 0.f;
      if (i < n) e = by_count ? 1.0f : __expf(okey_to_float(~(uint32_t)(keys[i] >> 32)) - M);
      float inc = e;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float a = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += a;
      }
      if (lane == 31) w_sum[warp] = inc;
      __syncthreads();
      float wbase = 0.f, tot = 0.f;
      for (int w = 0; w < kFinWarps; ++w) {
        if (w < warp) wbase += w_sum[w];
        tot += w_sum[w];
      }
      const float cum = above + s_run + wbase + inc;
      if (i < n && cum >= target) atomicMin(&s_pick, i);
      __syncthreads();
      if (i == s_pick) s_pick_mass = cum;
      if (tid == 0) s_run += tot;
      __syncthreads();
    }
    int pick = s_pick;
    float mass = s_pick_mass;
    if (pick == kNoPick) {
      pick = n - 1;
      mass = above + s_run;
    }
    if (pick < 0) pick = 0;  // n == 0 cannot happen (bucket holds >= 1 key)
    const int c = pick + 1;
    if (ids) {
      for (int i = tid; i < c; i += kFinThreads) {
        const int pos = emit_base + i;
        if (pos < sel_stride) ids[pos] = (int)(uint32_t)keys[i];
      }
    }
    const uint32_t thr_key = ~(uint32_t)(keys[pick] >> 32);
    const int thr_last = (int)(uint32_t)keys[pick];
    const int extra = add_forced(thr_key, thr_last, base + c, mass);
    if (tid == 0) {
      sel_count[rh] = base + c + extra;
      if (sel_mass) sel_mass[rh] = mass / Z;
      if (sel_thresh) sel_thresh[rh] = okey_to_float(thr_key);
      if (sel_tie_last) sel_tie_last[rh] = thr_last;
      if (ids && base + c + extra > sel_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }

  if (tie) {
    // More than kCandCap keys share the threshold score exactly: take the first c of them in
    // position order, c = the number of equal masses still needed.
    const uint32_t t_key = tie_key;
    const float e_t = by_count ? 1.0f : __expf(okey_to_float(t_key) - M);
    int c = (int)ceilf((target - above) / e_t);
    c = max(1, min(c, tie_bucket));
    if (tid == 0) {
      s_emitted = 0;
      s_last = -1;
    }
    __syncthreads();
    const int n_pages = (n_keys + kPage - 1) >> kPageShift;
    for (int p0 = 0; p0 < n_pages; p0 += kFinWarps) {
      if (s_emitted >= c) break;  // uniform (see barrier at the end of the round)
      // ordered emission: thread t owns keys 2t, 2t+1 of this round
      const int n_first = p0 * kPage + 2 * tid;
      int f0 = 0, f1 = 0;
      if (n_first < n_keys) {
        const float2 sv = *reinterpret_cast<const float2*>(row + n_first);
        f0 = okey(sv.x) == t_key;
        f1 = n_first + 1 < n_keys && okey(sv.y) == t_key;
      }
      int inc = f0 + f1;
      const int mine = inc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += a;
      }
      if (lane == 31) w_cnt[warp] = inc;
      __syncthreads();
      int wbase = 0, tot = 0;
      for (int w = 0; w < kFinWarps; ++w) {
        if (w < warp) wbase += w_cnt[w];
        tot += w_cnt[w];
      }
      int before = s_emitted + wbase + inc - mine;
      if (f0) {
        if (before < c) {
          if (ids && emit_base + before < sel_stride) ids[emit_base + before] = n_first;
          atomicMax(&s_last, n_first);
        }
        ++before;
      }
      if (f1 && before < c) {
        if (ids && emit_base + before < sel_stride) ids[emit_base + before] = n_first + 1;
        atomicMax(&s_last, n_first + 1);
      }
      __syncthreads();
      if (tid == 0) s_emitted += tot;
      __syncthreads();
    }
    float mass = above + (float)c * e_t;
    const int t_last = s_last;
    const int extra = add_forced(t_key, t_last, base + c, mass);
    if (tid == 0) {
      sel_count[rh] = base + c + extra;
      if (sel_mass) sel_mass[rh] = mass / Z;
      if (sel_thresh) sel_thresh[rh] = okey_to_float(t_key);
      if (sel_tie_last) sel_tie_last[rh] = t_last;
      if (ids && base + c + extra > sel_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }
  // still refining after every level: cannot happen (three levels resolve all 32 key bits)
  if (tid == 0) {
    sel_count[rh] = 0;
    set_status(status, RTP_ERR_UNSUPPORTED);
  }
}

__global__ void __launch_bounds__(kFinThreads) sel_finalize_kernel(
    const Dims d, const float* __restrict__ scores, const int64_t l_pad, SelState* __restrict__ state,
    const uint2* __restrict__ cand, const int list_cap, int32_t* __restrict__ sel_idx, int64_t sel_stride,
    int32_t* __restrict__ sel_count,
    float* __restrict__ sel_mass, float* __restrict__ sel_thresh, int32_t* __restrict__ sel_tie_last,
    int32_t* status) {
  chain_wait();
  extern __shared__ __align__(16) unsigned char fin_smem[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(fin_smem);       // [kCandCap] candidates
  unsigned long long* keys2 = keys + kCandCap;                                       // [kCandCap] the other buffer
  const int64_t rh = blockIdx.x;
  finalize_core(d, scores + rh * l_pad, state + rh, cand + rh * (int64_t)list_cap, list_cap, false, keys, keys2, rh, sel_idx,
                sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status);
}

// ---- short contexts: the whole selection of a (row, head) in one CTA ------------------------------------------------
// When the scores of a row fit into shared memory, one CTA of kFinThreads threads scores the row's keys for its head,
// keeps the scores on chip and runs every later step on them (level-1 histogram, key levels, compaction, finish): one
// launch instead of six, no pass over global memory after the scan.  The index keys of an index head are read by each
// of its heads' CTAs (they mostly come from the L2 cache).  The arithmetic is that of the general path: the same bin
// functions, the same resolves (l1_resolve_warp, key_resolve_warp) and the same finish (finalize_core).
// Measured against the general path (B = 8, call time of the selection): 33 against 58 us at 2K keys, 36 against 59 at 4K,
// 41 against 54 at 8K; with its own scan 50 against 56 at 16K and 71 against 59 at 32K (the heads of an index head each
// score all of its keys); with the scan shared (SCAN = false) 41 against 55 at 16K and 52 against 57 at 32K.
constexpr int kSmallMaxKeys = 8192;    // own scan: 32 KB of scores beside the two candidate buffers of the finish (64 KB)
constexpr int kMidMaxKeys = 36864;     // with stored scores: 144 KB of them in shared memory

// SCAN = false: the scores were stored by sel_score_kernel (all SMs share the scan); the CTA copies its row into shared
// memory instead of scoring it (used between 8K and 36K keys, where one CTA's own scan is the slower way).
template <bool NH4, bool F8, bool SCAN>
__global__ void __launch_bounds__(kFinThreads) sel_small_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows, const __nv_bfloat16* __restrict__ qt,
    const float* __restrict__ stored, const int64_t l_pad, int32_t* __restrict__ sel_idx, int64_t sel_stride, int32_t* __restrict__ sel_count, float* __restrict__ sel_mass,
    float* __restrict__ sel_thresh, int32_t* __restrict__ sel_tie_last, int32_t* status) {
  chain_wait();
  extern __shared__ __align__(16) unsigned char fin_smem[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(fin_smem);
  unsigned long long* keys2 = keys + kCandCap;
  float* sc = reinterpret_cast<float*>(fin_smem + 2 * kCandCap * sizeof(unsigned long long));   // the row's scores
  uint32_t* hw = reinterpret_cast<uint32_t*>(keys2);   // [kFinWarps][kBins] level-1 sums per warp (before the finish needs keys2)
  __shared__ SelState s_st;
  __shared__ uint32_t h1[kBins][3];   // key levels: {sum, carries, count} per bin
  __shared__ uint32_t w_key[kFinWarps];
  __shared__ int s_n_above, s_n_in;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t rh = blockIdx.x;
  const int64_t r = rh / d.n_ret;
  const int i_ret = (int)(rh % d.n_ret);
  const int ih = hm.q2ih[i_ret], slot = hm.slot_in_ih[i_ret], nh = hm.ih_nheads[ih];
  const int seq = rows.row_seq(r);
  int n_keys = rows.row_pos(r) + 1;
  {
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;   // (never beyond the block table)
    if (n_keys > sl) {
      if (tid == 0) set_status(status, RTP_ERR_INVALID);
      n_keys = sl;
    }
    n_keys = max(0, n_keys);
  }
  const int n_pages = (n_keys + kPage - 1) >> kPageShift;
  const bool by_count = d.top_k > 0;
  int32_t* ids = sel_idx ? sel_idx + rh * sel_stride : nullptr;

  // ---- the scan: a warp scores a page for the index head's heads (MMA) and keeps this head's scores ----
  float mx = -INFINITY;
  if (!SCAN) {
    const float* src = stored + rh * l_pad;
    for (int n4 = 4 * tid; n4 < n_pages * kPage; n4 += 4 * kFinThreads) {
      const float4 v = ld_scores4(src + n4);
      *reinterpret_cast<float4*>(sc + n4) = v;
      if (n4 < n_keys) mx = fmaxf(mx, v.x);
      if (n4 + 1 < n_keys) mx = fmaxf(mx, v.y);
      if (n4 + 2 < n_keys) mx = fmaxf(mx, v.z);
      if (n4 + 3 < n_keys) mx = fmaxf(mx, v.w);
    }
  } else {
    RowCtx x;
    x.r = r; x.ih = ih; x.split = 0; x.seq = seq; x.n_keys = n_keys; x.p_lo = 0; x.p_hi = n_pages; x.nh = nh;
    QFrag qf = load_qfrag(qt + r * d.n_ret * kIndexDim, hm.ih_heads[ih], nh, lane);
    if (F8 && !qfrag_to_f16(qf)) set_status(status, RTP_ERR_UNSUPPORTED);   // a projected query beyond fp16's range
    const int g = lane >> 2;
    const bool mine = NH4 ? (g & 3) == slot : g == (slot & 7);
    const int e_lo = NH4 ? 0 : (slot < 8 ? 0 : 4), e_hi = NH4 ? 2 : e_lo + 4;
    uint4 v[4], vn[4], vnn[4];   // two pages in flight ahead of the one that is scored
    if (warp < n_pages) load_page<F8>(cv, x, warp, lane, vn);
    if (warp + kFinWarps < n_pages) load_page<F8>(cv, x, warp + kFinWarps, lane, vnn);
    for (int p = warp; p < n_pages; p += kFinWarps) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[i] = vn[i];
        vn[i] = vnn[i];
      }
      if (p + 2 * kFinWarps < n_pages) load_page<F8>(cv, x, p + 2 * kFinWarps, lane, vnn);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float s_lo[4], s_hi[4];
        if (F8) score16_f8(qf, make_uint2(v[i].x, v[i].y), lane, s_lo, s_hi); else score16(qf, v[i], lane, s_lo, s_hi);
        const LaneElems<NH4> el = lane_elems<NH4>(s_lo, s_hi, lane);
        if (mine) {
#pragma unroll
          for (int e = 0; e < LaneElems<NH4>::kN; ++e) {
            if (e < e_lo || e >= e_hi) continue;
            const int n = p * kPage + i * 16 + el.koff[e];
            const float sv = finish_score(el.raw[e], d.score_scale);
            sc[n] = sv;   // (entries of the last page beyond the row's keys are written and never read)
            if (n < n_keys) mx = fmaxf(mx, sv);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) w_key[warp] = okey(mx + 0.0f);
  for (int i = tid; i < kFinWarps * kBins; i += kFinThreads) hw[i] = 0u;
  if (tid == 0) {
    SelState z = {};
    z.n_keys = n_keys;
    const bool every = by_count ? d.top_k >= n_keys : d.top_p >= 1.0f;
    z.mode = (every || n_keys <= 1) ? kSelectAll : kRefine;
    z.hi_key = 0xffffffffu;
    s_st = z;
  }
  __syncthreads();
  uint32_t kmax = 0u;
  for (int w = 0; w < kFinWarps; ++w) kmax = max(kmax, w_key[w]);
  const float M = l1_anchor(okey_to_float(kmax));   // the reference of the histograms: the maximum rounded up

  if (s_st.mode == kRefine) {   // (uniform)
    // ---- level 1: mass histogram over M - s, one private copy per warp (2^17 fixed point, no wait per add) ----
    for (int n = tid; n < n_keys; n += kFinThreads) {
      const float sv = sc[n];
      float bin_f;
      const int bin = l1_bin_f(M, sv, bin_f);
      const float arg = l1_mass_arg(M, sv, bin_f);
      add_mass17(&hw[warp * kBins + bin], by_count ? 20.0f : arg);
    }
    __syncthreads();
    if (warp == 0) {
      unsigned long long u0 = 0ull, u1 = 0ull;
      for (int w = 0; w < kFinWarps; ++w) {
        u0 += (unsigned long long)hw[w * kBins + 2 * lane] << 3;       // back to the 2^20 scale of the resolve
        u1 += (unsigned long long)hw[w * kBins + 2 * lane + 1] << 3;
      }
      l1_resolve_warp(d, M, __ull2float_rn(u0), __ull2float_rn(u1), u0 != 0ull, u1 != 0ull, lane, kCandCap, &s_st, status);
    }
    __syncthreads();
    // ---- key levels: six more key bits inside the bucket, with exact counts, until it holds at most kCandCap keys ----
#pragma unroll 1
    for (int level = 0; level < 7 && s_st.mode == kRefine; ++level) {
      for (int i = tid; i < kBins * 3; i += kFinThreads) (&h1[0][0])[i] = 0u;
      __syncthreads();
      const uint32_t lo_key = s_st.lo_key, span = s_st.span;
      const int shift = s_st.shift;
      const float ref_s = s_st.ref_s, lw = by_count ? 0.f : kLog2eH;
      for (int n = tid; n < n_keys; n += kFinThreads) {
        const float sv = sc[n];
        const uint32_t t = okey(sv) - lo_key;
        if (t < span) {
          uint32_t* acc = &h1[t >> shift][0];
          add_mass(acc, fmaf(sv - ref_s, lw, 20.0f));
          atomicAdd(acc + 2, 1u);
        }
      }
      __syncthreads();
      if (warp == 0) {
        const int b0 = 63 - 2 * lane, b1 = 62 - 2 * lane;
        key_resolve_warp(d, acc_mass(h1[b0][0], h1[b0][1]), acc_mass(h1[b1][0], h1[b1][1]), h1[b0][2], h1[b1][2], lane,
                         kCandCap, &s_st, status);
      }
      __syncthreads();
    }
  }

  // ---- compaction: keys above the bucket are emitted, keys inside it become the candidates of the finish ----
  {
    const int mode = s_st.mode;
    const bool all = mode == kSelectAll, bucket = mode == kCollect || mode == kTieScan, collect = mode == kCollect;
    const uint32_t lo_key = s_st.lo_key, hi_key = s_st.hi_key;
    const uint32_t lt = (1u << lane) - 1u;
    if (tid == 0) {
      s_n_above = 0;
      s_n_in = 0;
    }
    __syncthreads();
    for (int n0 = 0; n0 < n_keys; n0 += kFinThreads) {
      const int n = n0 + tid;
      const bool ok = n < n_keys;
      const uint32_t key = ok ? okey(sc[n]) : 0u;
      const bool fa = ok && (all || (bucket && key > hi_key));
      const bool fc = ok && collect && key >= lo_key && key <= hi_key;
      const uint32_t ma = __ballot_sync(0xffffffffu, fa);
      if (ma) {
        int base = 0;
        if (lane == 0) base = atomicAdd(&s_n_above, __popc(ma));
        base = __shfl_sync(0xffffffffu, base, 0);
        const int pos = base + __popc(ma & lt);
        if (fa && ids && pos < sel_stride) ids[pos] = n;
      }
      const uint32_t mc = __ballot_sync(0xffffffffu, fc);
      if (mc) {
        int base = 0;
        if (lane == 0) base = atomicAdd(&s_n_in, __popc(mc));
        base = __shfl_sync(0xffffffffu, base, 0);
        const int pos = base + __popc(mc & lt);
        if (fc && pos < kCandCap) keys[pos] = ((unsigned long long)(~key) << 32) | (unsigned long long)(uint32_t)n;
      }
    }
    __syncthreads();
    if (tid == 0 && !all) {
      s_st.cnt_above = s_n_above;
      s_st.emit_cnt = ids ? s_n_above : 0;
      s_st.cand_cnt = min(s_n_in, kCandCap);
      if (collect) s_st.bucket_cnt = s_n_in;
    }
    __syncthreads();
  }
  finalize_core(d, sc, &s_st, nullptr, kCandCap, true, keys, keys2, rh, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh,
                sel_tie_last, status);
}

int select_splits(const Dims& d, int64_t R, int64_t max_len, int sm_count) {
  const int64_t pages = (max_len + kPage - 1) / kPage;
  int64_t want = (4LL * sm_count + R * d.n_ih - 1) / (R * d.n_ih);
  int64_t cap = (pages + 31) / 32;  // at least 32 pages (2048 keys) per CTA
  int64_t s = want < cap ? want : cap;
  const int64_t least = (pages + 2047) / 2048;   // at most 2048 pages per CTA = 16384 keys per warp (32-bit bin sums)
  if (s < least) s = least;
  if (s < 1) s = 1;
  if (s > 4096) s = 4096;
  return (int)s;
}

struct SelWorkspace {
  SelState* state;
  unsigned long long* g_mass;   // [row heads][64] merged bin sums
  uint32_t* g_cnt;              // [row heads][64] merged bin counts
  uint32_t* tickets;            // [rows * index heads]
  uint2* cand;
  float* scores;                // [row heads][l_pad] scores of the first pass
  size_t zero_off, zero_bytes;  // the part that must be zero before the first pass
  size_t bytes;
};

constexpr int kListCap = 65536;   // candidates per (row, head) kept in global memory (never more than the padded length)
int list_capacity(int64_t l_pad) { return (int)(l_pad < kListCap ? l_pad : kListCap); }

SelWorkspace carve(void* ws, int64_t n_rowheads, int64_t n_units, int64_t l_pad) {
  SelWorkspace w;
  size_t off = 0;
  auto take = [&](size_t n) {
    size_t o = off;
    off += (n + 255) & ~(size_t)255;
    return o;
  };
  const size_t o_state = take(sizeof(SelState) * n_rowheads);
  const size_t o_mass = take(sizeof(unsigned long long) * kBins * n_rowheads);
  const size_t o_cnt = take(sizeof(uint32_t) * kBins * n_rowheads);
  const size_t o_tick = take(sizeof(uint32_t) * n_units);
  const size_t o_cand = take(sizeof(uint2) * (size_t)list_capacity(l_pad) * n_rowheads);
  const size_t o_scores = take(sizeof(float) * (size_t)l_pad * n_rowheads);
  char* b = reinterpret_cast<char*>(ws);
  w.state = reinterpret_cast<SelState*>(b + o_state);
  w.g_mass = reinterpret_cast<unsigned long long*>(b + o_mass);
  w.g_cnt = reinterpret_cast<uint32_t*>(b + o_cnt);
  w.tickets = reinterpret_cast<uint32_t*>(b + o_tick);
  w.cand = reinterpret_cast<uint2*>(b + o_cand);
  w.scores = reinterpret_cast<float*>(b + o_scores);
  w.zero_off = o_mass;
  w.zero_bytes = o_cand - o_mass;
  w.bytes = off;
  return w;
}

constexpr int kKeyLevels = 6;   // 6 bits each: a level-1 bucket spans fewer than 2^32 key values

}  // namespace

int64_t padded_len(int64_t max_len) { return (max_len + kPage - 1) / kPage * kPage; }

size_t select_rows_workspace_bytes(const Dims& d, int64_t R, int64_t max_len) {
  if (R <= 0 || d.n_ret <= 0) return 0;
  return carve(nullptr, R * d.n_ret, R * d.n_ih, padded_len(max_len)).bytes;
}

cudaError_t launch_select_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const __nv_bfloat16* qt, int64_t max_len, int32_t* sel_idx, int64_t sel_stride,
                               int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                               int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  const int64_t nrh = rows.R * d.n_ret;
  const int64_t l_pad = padded_len(max_len);
  int max_nh = 0;
  for (int i = 0; i < d.n_ih; ++i) max_nh = hm.ih_nheads[i] > max_nh ? hm.ih_nheads[i] : max_nh;
  const bool one_cta = d.select_path != 1 && nrh <= 2LL * sm_count;
  if (one_cta && l_pad <= kSmallMaxKeys) {
    // short contexts: one CTA per (row, head) does everything on chip
    const int smem = 2 * kCandCap * 8 + (int)l_pad * 4;
    cudaError_t es = cudaSuccess;
#define RTP_SMALL(NH4_, F8_)                                                                                              \
  {                                                                                                                       \
    static PerDeviceOnce once;                                                                                            \
    es = set_dyn_smem_once(sel_small_kernel<NH4_, F8_, true>, 2 * kCandCap * 8 + kSmallMaxKeys * 4, once);                \
    if (es == cudaSuccess)                                                                                                \
      (void)launch_chained(sel_small_kernel<NH4_, F8_, true>, dim3((unsigned)nrh), dim3(kFinThreads), (size_t)smem, st, cv, d, hm, \
                           rows, qt, nullptr, l_pad, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status); \
  }
    if (max_nh <= 4) {
      if (cv.ikey_fp8) RTP_SMALL(true, true) else RTP_SMALL(true, false)
    } else {
      if (cv.ikey_fp8) RTP_SMALL(false, true) else RTP_SMALL(false, false)
    }
#undef RTP_SMALL
    return es != cudaSuccess ? es : cudaGetLastError();
  }
  const SelWorkspace w = carve(ws, nrh, rows.R * d.n_ih, l_pad);
  const int list_cap = list_capacity(l_pad);
  cudaError_t e = cudaSuccess;
  const bool mid = one_cta && l_pad <= kMidMaxKeys;   // (its last kernel keeps the selection state on chip: nothing to reset)
  if (!mid) {
    const int64_t n_zero = (int64_t)(w.zero_bytes / 4);
    const int64_t work = n_zero > nrh ? n_zero : nrh;
    const int64_t cap_blocks = (int64_t)sm_count * 8;
    const unsigned blocks = (unsigned)((work + 255) / 256 < cap_blocks ? (work + 255) / 256 : cap_blocks);
    (void)launch_chained(sel_init_kernel, dim3(blocks), dim3(256), 0, st, cv, d, rows, w.state, nrh,
                                            reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(ws) + w.zero_off), n_zero);
  }
  const int n_splits = select_splits(d, rows.R, max_len, sm_count);
  const dim3 grid((unsigned)(rows.R * d.n_ih), n_splits);
  // one scan of the index keys (scores stored, row maxima), then three passes over the stored scores
#define RTP_SCORE(NH4_, F8_) \
  (void)launch_chained(sel_score_kernel<NH4_, F8_>, dim3(grid), dim3(kThreads), 0, st, cv, d, hm, rows, qt, w.state, w.scores, l_pad, n_splits, status)
  if (max_nh <= 4) {
    if (cv.ikey_fp8) RTP_SCORE(true, true); else RTP_SCORE(true, false);
  } else {
    if (cv.ikey_fp8) RTP_SCORE(false, true); else RTP_SCORE(false, false);
  }
#undef RTP_SCORE
  if (mid) {
    // medium contexts: the scan above is shared by all SMs; one CTA per (row, head) takes its stored scores on chip and
    // does the rest (the state written by the kernels above is not used)
    static PerDeviceOnce once;
    e = set_dyn_smem_once(sel_small_kernel<true, false, false>, 2 * kCandCap * 8 + kMidMaxKeys * 4, once);
    if (e != cudaSuccess) return e;
    (void)launch_chained(sel_small_kernel<true, false, false>, dim3((unsigned)nrh), dim3(kFinThreads),
                         (size_t)(2 * kCandCap * 8 + (int)l_pad * 4), st, cv, d, hm, rows, qt, w.scores, l_pad, sel_idx, sel_stride,
                         sel_count, sel_mass, sel_thresh, sel_tie_last, status);
    return cudaGetLastError();
  }
  (void)launch_chained(sel_l1_kernel, dim3(grid), dim3(kThreads), 0, st, cv, d, hm, rows, w.scores, l_pad, w.state, w.g_mass, w.tickets, n_splits, list_cap, status);
  (void)launch_chained(sel_key_kernel, dim3(grid), dim3(kThreads), 0, st, cv, d, hm, rows, w.scores, l_pad, w.state, w.g_mass, w.g_cnt, w.tickets,
                                            n_splits, 1 + kKeyLevels, list_cap, status);
  {
    const dim3 grid3((unsigned)(rows.R * d.n_ih), n_splits, (max_nh + kHeadsPerCta - 1) / kHeadsPerCta);
    (void)launch_chained(sel_compact_kernel, dim3(grid3), dim3(kThreads), 0, st, cv, d, hm, rows, w.scores, l_pad, w.state, w.cand, list_cap, sel_idx,
                                                   sel_stride, n_splits, status);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  constexpr int kFinSmem = 2 * kCandCap * 8;
  static PerDeviceOnce fin_once;
  e = set_dyn_smem_once(sel_finalize_kernel, kFinSmem, fin_once);
  if (e != cudaSuccess) return e;
  (void)launch_chained(sel_finalize_kernel, dim3((unsigned)nrh), dim3(kFinThreads), kFinSmem, st, d, w.scores, l_pad, w.state, w.cand, list_cap, sel_idx, sel_stride,
                                                             sel_count, sel_mass, sel_thresh, sel_tie_last, status);
  return cudaGetLastError();
}

}  // namespace rtp
