// S2-S4 for a prefill chunk: fused indexer + top-p selection (Eq. 5) for rows q_start .. q_start+C-1
// of one sequence.
//
// A CTA owns 128 (row, head) pairs: (128 / G) consecutive positions x the G retrieval heads of one
// index head; each warp owns 16 of them (one head, 16 positions).  The CTA streams the index keys
// 0 .. last position (2 KB per page, cp.async double buffer) once per pass; a warp scores a 64-key
// page against its 16 rows with eight m16n8k16 MMAs.  All selection state lives in shared memory, so
// the whole selection of the chunk is one kernel without inter-CTA communication:
//   pass 0   row maximum M                                            (1 op per score)
//   pass 1   128-bin histogram of softmax mass over d = M - s in steps of 1/4 (d >= 31.75 pooled);
//            gives Z and the bucket in which the cumulative mass reaches p * Z; the bucket is then
//            turned into the exact interval of ordered score keys that fall into it (bisection)
//   pass 2+  64-bin (mass, count) histograms of the ordered key inside the interval, 6 key bits per
//            pass, until the interval holds one key or a single key value
//   tie pass only when equal scores straddle the cut: position of the last tie taken
// Rows drop out as soon as they are resolved; the CTA stops when all its rows are.  When id lists
// are requested, one more sweep appends every row's members in position order.
// Each pass has its own inner loop; pages that lie wholly below a warp's first row need no causal test.
#include <cstdlib>
#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kCWarps = 8;
constexpr int kCThreads = kCWarps * 32;
constexpr int kCRows = 128;
constexpr int kPagesPerStage = 4;
constexpr int kStageKeys = kPagesPerStage * kPage;                  // 256 keys
constexpr int kStageBytesC = kStageKeys * kIndexDim * 2;            // 8 KB
constexpr int kL1Bins = 128;
constexpr float kL1Scale = 4.0f;                                    // bins per unit of d
constexpr int kSubBins = 64;
constexpr int kMaxPasses = 12;
constexpr float kLog2eC = 1.4426950408889634f;

enum Phase { kPhMax = 0, kPhL1 = 1, kPhKey = 2, kPhTie = 3, kPhDone = 4 };

struct RowState {      // one per (row, head), in shared memory
  float M, Z, target, mass_above;
  uint32_t base_key;   // key levels: bucket = keys in [base_key, base_key + span)
  uint32_t span;
  int32_t shift;       // bin = (key - base_key) >> shift, in [0, 64)
  uint32_t hi_count;   // first key level: keys > hi_count are counted as "above the bucket"; else 0xffffffff
  int32_t phase;
  int32_t cnt_above;   // keys strictly above the current bucket
  int32_t tie_need;    // tie pass: number of ties to take
  uint32_t thr_key;    // result: selected <=> key > thr_key or (key == thr_key and n <= tie_last)
  int32_t tie_last;
  int32_t n_keys;
  float sel_mass;
  int32_t count;
  float raw_lo, raw_hi;   // raw-value interval of the current key bucket
  float raw_hic;          // first key level: raw values above this lie above the bucket; else +inf
  float tie_lo, tie_hi;   // raw-value interval of thr_key (tie pass)
};

constexpr int kHistBytes = kCRows * kL1Bins * 4;                    // 64 KB (key levels reuse it as 64 x {mass,cnt})
constexpr int kSmemC = kHistBytes + 2 * kStageBytesC + kCRows * (int)sizeof(RowState);

__device__ __forceinline__ void cp_async16c(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ uint32_t smem_u32c(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Level-1 bin of a score: the same arithmetic in the histogram pass and in the bisection below.
__device__ __forceinline__ int l1_bin(float M, float s) {
  return min(kL1Bins - 1, (int)((M - s) * kL1Scale));
}

// Per-lane view of its two rows for one pass (registers).
struct LaneRows {
  float M_a, M_b;
  uint32_t base_a, base_b;
  int shift_a, shift_b;
  int pos_a, pos_b;
  // Unscaled MMA outputs are compared directly: the keys of a bucket are the images of one closed interval of
  // raw values (finish_score is monotone), found by bisection when the bucket is chosen.
  float lo_a, hi_a, lo_b, hi_b;      // raw interval of the current key bucket (empty: lo = +inf, hi = -inf)
  float hic_a, hic_b;                // raw values above this are counted as "above the bucket" (+inf: none)
  float tlo_a, thi_a, tlo_b, thi_b;  // raw interval of the tied key value (tie pass)
};

// ---- one 64-key page, one warp ----------------------------------------------------------------------
template <bool MASK>
__device__ __forceinline__ void page_max(const unsigned char* pg, const QFrag& iq, int lane, int n_page,
                                         const LaneRows& L, float& mx_a, float& mx_b) {
  const int g = lane >> 2, c = lane & 3;
  const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const uint2 b = *reinterpret_cast<const uint2*>(pg + (nt * 8 + g) * (kIndexDim * 2) + boff);
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
    float s4[4];
    mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
    if (MASK) {
      const int n0 = n_page + nt * 8 + 2 * c;
      if (n0 > L.pos_a) s4[0] = -INFINITY;
      if (n0 + 1 > L.pos_a) s4[1] = -INFINITY;
      if (n0 > L.pos_b) s4[2] = -INFINITY;
      if (n0 + 1 > L.pos_b) s4[3] = -INFINITY;
    }
    mx_a = fmaxf(mx_a, fmaxf(s4[0], s4[1]));
    mx_b = fmaxf(mx_b, fmaxf(s4[2], s4[3]));
  }
}

template <bool MASK>
__device__ __forceinline__ void page_l1(const unsigned char* pg, const QFrag& iq, int lane, int n_page,
                                        const LaneRows& L, float scale, float* hist_a, float* hist_b) {
  const int g = lane >> 2, c = lane & 3;
  const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const uint2 b = *reinterpret_cast<const uint2*>(pg + (nt * 8 + g) * (kIndexDim * 2) + boff);
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
    float s4[4];
    mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
    const int n0 = n_page + nt * 8 + 2 * c;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool lo = e < 2;
      if (MASK && n0 + (e & 1) > (lo ? L.pos_a : L.pos_b)) continue;
      const float s = finish_score(s4[e], scale);
      const float dd = (lo ? L.M_a : L.M_b) - s;
      const int bin = max(0, min(kL1Bins - 1, (int)(dd * kL1Scale)));   // (rows that are already done have no M)
      atomicAdd((lo ? hist_a : hist_b) + bin, fast_ex2(-dd * kLog2eC));
    }
  }
}

// Key levels (and, when TIE, the in-order tie count).  Rows that are not in a key level carry span = 0 and
// hic = 0xffffffff, rows that are not in the tie pass carry need = 0, so no per-row branching is needed.
template <bool MASK, bool TIE>
__device__ __forceinline__ void page_late(const unsigned char* pg, const QFrag& iq, int lane, int n_page,
                                          const LaneRows& L, float scale, float* hist_a, float* hist_b,
                                          int& cnt_a, int& cnt_b, int need_a, int need_b,
                                          int& run_a, int& run_b, int& tl_a, int& tl_b) {
  const int g = lane >> 2, c = lane & 3;
  const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const uint2 b = *reinterpret_cast<const uint2*>(pg + (nt * 8 + g) * (kIndexDim * 2) + boff);
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
    float s4[4];
    mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
    const int n0 = n_page + nt * 8 + 2 * c;
    int tf_a = 0, tf_b = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool lo = e < 2;
      float raw = s4[e];
      if (MASK && n0 + (e & 1) > (lo ? L.pos_a : L.pos_b)) raw = __int_as_float(0x7fc00000);   // NaN: fails every test
      if (raw >= (lo ? L.lo_a : L.lo_b) && raw <= (lo ? L.hi_a : L.hi_b)) {
        const float s = finish_score(raw, scale);
        const uint32_t t = okey(s) - (lo ? L.base_a : L.base_b);
        float* h = (lo ? hist_a : hist_b) + 2 * (t >> (lo ? L.shift_a : L.shift_b));
        atomicAdd(h, fast_ex2((s - (lo ? L.M_a : L.M_b)) * kLog2eC));
        atomicAdd(reinterpret_cast<int*>(h + 1), 1);
      } else if (raw > (lo ? L.hic_a : L.hic_b)) {
        if (lo) ++cnt_a; else ++cnt_b;
      }
      if (TIE) {
        if (raw >= (lo ? L.tlo_a : L.tlo_b) && raw <= (lo ? L.thi_a : L.thi_b)) {
          if (lo) tf_a |= 1 << (e & 1); else tf_b |= 1 << (e & 1);
        }
      }
    }
    if (TIE) {
      // in-order prefix of the tied keys inside the quad (lane c holds keys 2c, 2c+1 of the n8 tile)
      const int ka = __popc(tf_a), kb = __popc(tf_b);
      int ia = ka, ib = kb, t;
      t = __shfl_up_sync(0xffffffffu, ia, 1, 4); if (c >= 1) ia += t;
      t = __shfl_up_sync(0xffffffffu, ia, 2, 4); if (c >= 2) ia += t;
      t = __shfl_up_sync(0xffffffffu, ib, 1, 4); if (c >= 1) ib += t;
      t = __shfl_up_sync(0xffffffffu, ib, 2, 4); if (c >= 2) ib += t;
      const int tot_a = __shfl_sync(0xffffffffu, ia, 3, 4), tot_b = __shfl_sync(0xffffffffu, ib, 3, 4);
      int before = run_a + ia - ka;
#pragma unroll
      for (int e = 0; e < 2; ++e)
        if (tf_a & (1 << e)) { if (before < need_a) tl_a = max(tl_a, n0 + e); ++before; }
      before = run_b + ib - kb;
#pragma unroll
      for (int e = 0; e < 2; ++e)
        if (tf_b & (1 << e)) { if (before < need_b) tl_b = max(tl_b, n0 + e); ++before; }
      run_a += tot_a;
      run_b += tot_b;
    }
  }
}

template <int G>
__global__ void __launch_bounds__(kCThreads, 2) select_chunk_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const __nv_bfloat16* __restrict__ qt,
    const int seq_id, const int q_start, const int C, int32_t* __restrict__ sel_idx, const int64_t sel_stride,
    int32_t* __restrict__ sel_count, float* __restrict__ sel_mass, float* __restrict__ sel_thresh,
    int32_t* __restrict__ sel_tie_last, int32_t* status, const int n_row_tiles, const int max_passes) {
  constexpr int BMP = kCRows / G;
  extern __shared__ __align__(128) unsigned char smem[];
  float* hist = reinterpret_cast<float*>(smem);                            // [128][128] floats
  unsigned char* stage_s = smem + kHistBytes;
  RowState* rs = reinterpret_cast<RowState*>(smem + kHistBytes + 2 * kStageBytesC);
  __shared__ int s_pending;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, c = lane & 3;
  const int tile = n_row_tiles - 1 - blockIdx.x;
  const int ih = blockIdx.y;
  const int nh = hm.ih_nheads[ih];
  const int r0 = tile * BMP;
  const int rows_here = min(BMP, C - r0);
  const int m0 = q_start + r0;
  const int seq_len = cv.seq_lens[seq_id];
  const int m_last = min(m0 + rows_here - 1, seq_len - 1);

  const int wrow = warp * 16;
  const int hslot = wrow / BMP, pofs = wrow % BMP;
  const bool warp_has_head = hslot < nh;
  const int rh_head = warp_has_head ? hm.ih_heads[ih][hslot] : 0;
  // the two rows of this lane: local ids la, lb in [0,128)
  const int la = wrow + g, lb = la + 8;
  const bool a_ok = warp_has_head && pofs + g < rows_here;
  const bool b_ok = warp_has_head && pofs + g + 8 < rows_here;
  const int pos_a = min(m0 + pofs + g, seq_len - 1), pos_b = min(m0 + pofs + g + 8, seq_len - 1);
  if (tid == 0 && m0 + rows_here - 1 >= seq_len) set_status(status, RTP_ERR_INVALID);
  const int warp_m_lo = min(m0 + pofs, seq_len - 1);
  const int warp_m_hi = min(m0 + pofs + 15, m_last);
  const bool warp_ok = warp_has_head && pofs < rows_here;

  // projected queries of the warp's rows
  QFrag iq = {0u, 0u, 0u, 0u};
  {
    const int off = qfrag_dim_offset(lane);
    if (a_ok) {
      const uint2 v = *reinterpret_cast<const uint2*>(qt + ((int64_t)(r0 + pofs + g) * d.n_ret + rh_head) * kIndexDim + off);
      iq.a0 = v.x;
      iq.a2 = v.y;
    }
    if (b_ok) {
      const uint2 v = *reinterpret_cast<const uint2*>(qt + ((int64_t)(r0 + pofs + g + 8) * d.n_ret + rh_head) * kIndexDim + off);
      iq.a1 = v.x;
      iq.a3 = v.y;
    }
  }
  if (tid < kCRows) {
    RowState z = {};
    const int hs = tid / BMP, po = tid % BMP;
    const bool ok = hs < nh && po < rows_here;
    z.n_keys = ok ? min(m0 + po, seq_len - 1) + 1 : 0;
    z.phase = ok && z.n_keys > 0 ? kPhMax : kPhDone;
    z.hi_count = 0xffffffffu;
    if (ok && z.n_keys > 0 && (d.top_p >= 1.0f || z.n_keys == 1)) {   // everything is selected
      z.phase = kPhDone;
      z.thr_key = 0u;
      z.tie_last = z.n_keys - 1;
      z.count = z.n_keys;
      z.sel_mass = 1.0f;
    }
    rs[tid] = z;
  }
  __syncthreads();

  const int n_pages = (m_last >> kPageShift) + 1;
  const int n_stages = (n_pages + kPagesPerStage - 1) / kPagesPerStage;
  const int64_t bt_base = (int64_t)seq_id * cv.max_pages;
  auto load_stage = [&](int sidx, int buf) {
    // 512 chunks of 16 bytes: page = chunk / 128
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      const int ch = tid + x * kCThreads;
      const int pg = sidx * kPagesPerStage + (ch >> 7);
      if (pg < n_pages) {
        const int phys = __ldg(cv.block_table + bt_base + pg);
        const __nv_bfloat16* src = cv.ikey + ((int64_t)phys * cv.n_ih + ih) * (kPage * kIndexDim) + (ch & 127) * 8;
        cp_async16c(smem_u32c(stage_s + buf * kStageBytesC + ch * 16), src);
      }
    }
  };

  const bool want_ids = sel_idx != nullptr;
  float* hist_a = hist + la * kL1Bins;
  float* hist_b = hist + lb * kL1Bins;
  const float scale = d.score_scale;

  for (int pass = 0; pass < max_passes; ++pass) {
    // ---- what does this pass do for my two rows? ----
    const RowState sa = rs[la], sb = rs[lb];
    const int ph_a = a_ok ? sa.phase : kPhDone, ph_b = b_ok ? sb.phase : kPhDone;
    if (tid == 0) s_pending = 0;
    for (int i = lane; i < 16 * kL1Bins; i += 32) hist[wrow * kL1Bins + i] = 0.f;   // this warp's histograms
    __syncthreads();
    const bool warp_active = __any_sync(0xffffffffu, ph_a != kPhDone || ph_b != kPhDone);
    // All rows of a warp do the max pass and the level-1 pass together; later passes mix key levels and ties.
    const bool pass_max = __any_sync(0xffffffffu, ph_a == kPhMax || ph_b == kPhMax);
    const bool pass_l1 = __any_sync(0xffffffffu, ph_a == kPhL1 || ph_b == kPhL1);
    const bool pass_tie = __any_sync(0xffffffffu, ph_a == kPhTie || ph_b == kPhTie);

    LaneRows LR;
    const float kInf = __int_as_float(0x7f800000);
    LR.M_a = sa.M; LR.M_b = sb.M;
    LR.pos_a = pos_a; LR.pos_b = pos_b;
    LR.base_a = sa.base_key; LR.base_b = sb.base_key;
    LR.shift_a = sa.shift; LR.shift_b = sb.shift;
    LR.lo_a = ph_a == kPhKey ? sa.raw_lo : kInf;  LR.hi_a = ph_a == kPhKey ? sa.raw_hi : -kInf;
    LR.lo_b = ph_b == kPhKey ? sb.raw_lo : kInf;  LR.hi_b = ph_b == kPhKey ? sb.raw_hi : -kInf;
    LR.hic_a = ph_a == kPhKey ? sa.raw_hic : kInf;
    LR.hic_b = ph_b == kPhKey ? sb.raw_hic : kInf;
    const bool tie_a = ph_a == kPhTie, tie_b = ph_b == kPhTie;
    LR.tlo_a = tie_a ? sa.tie_lo : kInf;  LR.thi_a = tie_a ? sa.tie_hi : -kInf;
    LR.tlo_b = tie_b ? sb.tie_lo : kInf;  LR.thi_b = tie_b ? sb.tie_hi : -kInf;
    const int need_a = tie_a ? sa.tie_need : 0, need_b = tie_b ? sb.tie_need : 0;

    float mx_a = -INFINITY, mx_b = -INFINITY;
    int cnt_a = 0, cnt_b = 0;
    int run_a = 0, run_b = 0;
    int tl_a = -1, tl_b = -1;

    load_stage(0, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int sidx = 0; sidx < n_stages; ++sidx) {
      const int buf = sidx & 1;
      if (sidx + 1 < n_stages) load_stage(sidx + 1, buf ^ 1);
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 1;" ::: "memory");
      __syncthreads();
      if (warp_active && warp_ok) {
        const unsigned char* st = stage_s + buf * kStageBytesC;
#pragma unroll 1
        for (int pg = 0; pg < kPagesPerStage; ++pg) {
          const int n_page = (sidx * kPagesPerStage + pg) * kPage;
          if (n_page > warp_m_hi) break;
          const unsigned char* pgp = st + pg * (kPage * kIndexDim * 2);
          const bool interior = n_page + kPage - 1 <= warp_m_lo;   // every key visible to every row of the warp
          if (pass_max) {
            if (interior) page_max<false>(pgp, iq, lane, n_page, LR, mx_a, mx_b);
            else page_max<true>(pgp, iq, lane, n_page, LR, mx_a, mx_b);
          } else if (pass_l1) {
            if (interior) page_l1<false>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b);
            else page_l1<true>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b);
          } else if (pass_tie) {
            if (interior) page_late<false, true>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b, cnt_a, cnt_b, need_a, need_b, run_a, run_b, tl_a, tl_b);
            else page_late<true, true>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b, cnt_a, cnt_b, need_a, need_b, run_a, run_b, tl_a, tl_b);
          } else {
            if (interior) page_late<false, false>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b, cnt_a, cnt_b, need_a, need_b, run_a, run_b, tl_a, tl_b);
            else page_late<true, false>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b, cnt_a, cnt_b, need_a, need_b, run_a, run_b, tl_a, tl_b);
          }
        }
      }
      __syncthreads();
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");

    // ---- end of pass: combine the quad's partial results ----
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
    cnt_a += __shfl_xor_sync(0xffffffffu, cnt_a, 1);
    cnt_a += __shfl_xor_sync(0xffffffffu, cnt_a, 2);
    cnt_b += __shfl_xor_sync(0xffffffffu, cnt_b, 1);
    cnt_b += __shfl_xor_sync(0xffffffffu, cnt_b, 2);
    tl_a = max(tl_a, __shfl_xor_sync(0xffffffffu, tl_a, 1));
    tl_a = max(tl_a, __shfl_xor_sync(0xffffffffu, tl_a, 2));
    tl_b = max(tl_b, __shfl_xor_sync(0xffffffffu, tl_b, 1));
    tl_b = max(tl_b, __shfl_xor_sync(0xffffffffu, tl_b, 2));
    __syncwarp();

    // Each of the warp's 16 rows is resolved by the whole warp in turn (bins spread over the lanes).
    // Every lane first copies the row state, then the warp synchronises, then one lane writes.
    for (int rr = 0; rr < 16; ++rr) {
      const int lr = wrow + rr;
      RowState* S = rs + lr;
      const RowState R = *S;
      __syncwarp();
      const int ph = R.phase;
      const int src_lane = (rr & 7) * 4;          // a lane of the quad that owns row rr
      const bool is_b = rr >= 8;
      if (ph == kPhDone || R.n_keys == 0) continue;
      if (ph == kPhMax) {
        // the maximum was taken on unscaled MMA outputs; scaling by a positive factor is monotone
        const float M = finish_score(__shfl_sync(0xffffffffu, is_b ? mx_b : mx_a, src_lane), scale);
        if (lane == 0) {
          S->M = M;
          S->phase = kPhL1;
        }
      } else if (ph == kPhL1) {
        // 128 bins, 4 per lane, bin 0 = highest scores
        float m4[4], tot = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          m4[k] = hist[lr * kL1Bins + lane * 4 + k];
          tot += m4[k];
        }
        float inc = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float tt = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += tt;
        }
        const float Z = __shfl_sync(0xffffffffu, inc, 31);
        const float target = d.top_p * Z * (1.0f + kMassMargin);
        int found = kL1Bins, lastb = -1;
        {
          float run = inc - tot;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if (m4[k] > 0.f) {
              lastb = lane * 4 + k;
              if (found == kL1Bins && run + m4[k] >= target) found = lane * 4 + k;
            }
            run += m4[k];
          }
        }
        int best = found;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lastb = max(lastb, __shfl_xor_sync(0xffffffffu, lastb, o));
        // rounding may leave the target just out of reach: then the lowest populated bin is the bucket
        if (best == kL1Bins) best = lastb;
        if (best >= 0 && (best >> 2) == lane) {
          float above = inc - tot;
          for (int k = 0; k < (best & 3); ++k) above += m4[k];
          S->Z = Z;
          S->target = target;
          S->mass_above = above;
          if (best == kL1Bins - 1) {
            // the cut falls into the pooled tail (mass below 2e-14 per key): take every key
            S->thr_key = 0u;
            S->tie_last = R.n_keys - 1;
            S->count = R.n_keys;
            S->sel_mass = 1.0f;
            S->phase = kPhDone;
          } else {
            // Exact interval [klo, khi] of ordered keys whose level-1 bin is `best`: l1_bin is monotone in the
            // key, so both ends are found by bisection between two keys that lie safely outside the bucket.
            const float M = R.M;
            const float hi_s = M - (float)best / kL1Scale, lo_s = M - (float)(best + 1) / kL1Scale;
            const float pad = 1e-5f * fmaxf(1.0f, fmaxf(fabsf(hi_s), fabsf(lo_s))) + 1e-3f;
            const uint32_t lo = okey(finish_score(lo_s - pad, 1.0f));
            const uint32_t hi = okey(finish_score(fminf(hi_s + pad, M), 1.0f));
            // klo = smallest key with bin <= best
            uint32_t a = lo, b2 = hi;            // invariant: bin(b2) <= best; bin(a) > best unless a is the answer
            if (l1_bin(M, okey_to_float(a)) <= best) b2 = a;
            while (a + 1 < b2) {
              const uint32_t mid = a + ((b2 - a) >> 1);
              if (l1_bin(M, okey_to_float(mid)) <= best) b2 = mid; else a = mid;
            }
            const uint32_t klo = b2;
            // khi = largest key with bin >= best
            a = klo; b2 = hi;                    // invariant: bin(a) >= best; bin(b2) < best unless b2 is the answer
            if (l1_bin(M, okey_to_float(b2)) >= best) a = b2;
            while (a + 1 < b2) {
              const uint32_t mid = a + ((b2 - a) >> 1);
              if (l1_bin(M, okey_to_float(mid)) >= best) a = mid; else b2 = mid;
            }
            const uint32_t khi = a;
            const uint32_t span = khi - klo + 1u;
            const int bits = span > 1u ? 32 - __clz(span - 1u) : 0;
            float rlo, rhi;
            raw_preimage(scale, klo, khi, rlo, rhi);
            S->base_key = klo;
            S->span = span;
            S->shift = max(0, bits - 6);
            S->hi_count = khi;
            S->raw_lo = rlo;
            S->raw_hi = rhi;
            S->raw_hic = rhi;
            S->cnt_above = 0;
            S->phase = kPhKey;
          }
        }
      } else if (ph == kPhKey) {
        // 64 bins of {mass, count}; bin 63 = highest keys.  Two bins per lane, lane 0 takes the top.
        const float* h = hist + lr * kL1Bins;
        const int bhi = 63 - 2 * lane, blo = bhi - 1;
        const float mh = h[2 * bhi], ml = h[2 * blo];
        const int ch = __float_as_int(h[2 * bhi + 1]), cl = __float_as_int(h[2 * blo + 1]);
        float incm = mh + ml;
        int incc = ch + cl;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float tm = __shfl_up_sync(0xffffffffu, incm, o);
          const int tc = __shfl_up_sync(0xffffffffu, incc, o);
          if (lane >= o) {
            incm += tm;
            incc += tc;
          }
        }
        const int extra_above = __shfl_sync(0xffffffffu, is_b ? cnt_b : cnt_a, src_lane);
        const float target = R.target;
        const float run = R.mass_above + incm - (mh + ml);
        const int runc = incc - (ch + cl);
        int found = -1, lowest = 64;
        if (ch > 0) {
          lowest = bhi;
          if (run + mh >= target) found = bhi;
        }
        if (cl > 0) {
          lowest = blo;
          if (found < 0 && run + mh + ml >= target) found = blo;
        }
        int best = found;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lowest = min(lowest, __shfl_xor_sync(0xffffffffu, lowest, o));
        if (best < 0) best = lowest;   // target out of reach by rounding: lowest populated bin
        if (best >= 64) {
          // empty bucket: cannot happen (the level-1 bucket holds at least one key)
          if (lane == 0) {
            S->phase = kPhDone;
            set_status(status, RTP_ERR_UNSUPPORTED);
          }
        } else if (best == bhi || best == blo) {
          const bool top = best == bhi;
          const float f_above = top ? run : run + mh;
          const int f_cnt_above = top ? runc : runc + ch;
          const int f_cnt = top ? ch : cl;
          const float f_mass = top ? mh : ml;
          const int shift = R.shift;
          const uint32_t ofs = (uint32_t)best << shift;
          const uint32_t lo_key = R.base_key + ofs;
          const uint32_t sub_span = min(1u << shift, R.span - ofs);
          const int cnt_above = R.cnt_above + extra_above + f_cnt_above;
          S->mass_above = f_above;
          S->cnt_above = cnt_above;
          float rlo, rhi;
          raw_preimage(scale, lo_key, lo_key + (sub_span - 1u), rlo, rhi);
          S->base_key = lo_key;
          S->span = sub_span;
          S->hi_count = 0xffffffffu;
          S->raw_lo = rlo;
          S->raw_hi = rhi;
          S->raw_hic = __int_as_float(0x7f800000);
          if (f_cnt == 1 || shift == 0) {
            // resolved: one key left, or a single key value (f_cnt equal scores)
            int take = f_cnt;
            if (f_cnt > 1) {
              const float each = f_mass / (float)f_cnt;
              take = (int)ceilf((target - f_above) / each);
              take = max(1, min(take, f_cnt));
            }
            S->thr_key = lo_key;
            S->count = cnt_above + take;
            S->sel_mass = (f_above + f_mass * ((float)take / (float)f_cnt)) / R.Z;
            if (take < f_cnt) {
              S->tie_need = take;
              S->tie_lo = rlo;   // shift == 0 here: the bucket is the single key value lo_key
              S->tie_hi = rhi;
              S->phase = kPhTie;
            } else {
              S->tie_last = R.n_keys - 1;
              S->phase = kPhDone;
            }
          } else {
            S->shift = max(0, shift - 6);
          }
        }
      } else if (ph == kPhTie) {
        const int tl = __shfl_sync(0xffffffffu, is_b ? tl_b : tl_a, src_lane);
        if (lane == 0) {
          S->tie_last = tl;
          S->phase = kPhDone;
        }
      }
    }
    __syncwarp();
    {
      int pend = 0;
      if (a_ok && rs[la].phase != kPhDone) pend = 1;
      if (b_ok && rs[lb].phase != kPhDone) pend = 1;
      if (pend) s_pending = 1;
    }
    __syncthreads();
    if (!s_pending) break;
    __syncthreads();
  }

  // ---- id lists: one more sweep over the keys, every resolved row appends its members in position order ----
  if (want_ids) {
    __syncthreads();
    const RowState sa = rs[la], sb = rs[lb];
    const bool em_a = a_ok && sa.phase == kPhDone && sa.n_keys > 0, em_b = b_ok && sb.phase == kPhDone && sb.n_keys > 0;
    int32_t* dst_a = sel_idx + ((int64_t)(r0 + pofs + g) * d.n_ret + rh_head) * sel_stride;
    int32_t* dst_b = sel_idx + ((int64_t)(r0 + pofs + g + 8) * d.n_ret + rh_head) * sel_stride;
    int run_a = 0, run_b = 0;
    load_stage(0, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int sidx = 0; sidx < n_stages; ++sidx) {
      const int buf = sidx & 1;
      if (sidx + 1 < n_stages) load_stage(sidx + 1, buf ^ 1);
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 1;" ::: "memory");
      __syncthreads();
      if (warp_ok) {
        const unsigned char* st = stage_s + buf * kStageBytesC;
        const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll 1
        for (int pg = 0; pg < kPagesPerStage; ++pg) {
          const int n_page = (sidx * kPagesPerStage + pg) * kPage;
          if (n_page > warp_m_hi) break;
#pragma unroll 1
          for (int nt = 0; nt < 8; ++nt) {
            const uint2 b = *reinterpret_cast<const uint2*>(st + (pg * kPage + nt * 8 + g) * (kIndexDim * 2) + boff);
            const float zero[4] = {0.f, 0.f, 0.f, 0.f};
            float s4[4];
            mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
            const int n_first = n_page + nt * 8 + 2 * c;
            int fa = 0, fb = 0;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int n = n_first + e;
              const uint32_t ka_ = okey(finish_score(s4[e], scale));
              const uint32_t kb_ = okey(finish_score(s4[2 + e], scale));
              if (em_a && n <= pos_a && (ka_ > sa.thr_key || (ka_ == sa.thr_key && n <= sa.tie_last))) fa |= 1 << e;
              if (em_b && n <= pos_b && (kb_ > sb.thr_key || (kb_ == sb.thr_key && n <= sb.tie_last))) fb |= 1 << e;
            }
            const int ka = __popc(fa), kb = __popc(fb);
            int ia = ka, ib = kb, tt;
            tt = __shfl_up_sync(0xffffffffu, ia, 1, 4); if (c >= 1) ia += tt;
            tt = __shfl_up_sync(0xffffffffu, ia, 2, 4); if (c >= 2) ia += tt;
            tt = __shfl_up_sync(0xffffffffu, ib, 1, 4); if (c >= 1) ib += tt;
            tt = __shfl_up_sync(0xffffffffu, ib, 2, 4); if (c >= 2) ib += tt;
            const int tot_a = __shfl_sync(0xffffffffu, ia, 3, 4), tot_b = __shfl_sync(0xffffffffu, ib, 3, 4);
            int wa = run_a + ia - ka, wb = run_b + ib - kb;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              if (fa & (1 << e)) { if (wa < sel_stride) dst_a[wa] = n_first + e; ++wa; }
              if (fb & (1 << e)) { if (wb < sel_stride) dst_b[wb] = n_first + e; ++wb; }
            }
            run_a += tot_a;
            run_b += tot_b;
          }
        }
      }
      __syncthreads();
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (c == 0) {
      if ((em_a && run_a > sel_stride) || (em_b && run_b > sel_stride)) set_status(status, RTP_ERR_CAPACITY);
    }
  }

  // ---- results ----
  if (tid < kCRows) {
    const int hs = tid / BMP, po = tid % BMP;
    if (hs < nh && po < rows_here) {
      const RowState& S = rs[tid];
      const int64_t o = (int64_t)(r0 + po) * d.n_ret + hm.ih_heads[ih][hs];
      if (S.phase != kPhDone) set_status(status, RTP_ERR_TIMEOUT);
      sel_count[o] = S.n_keys == 0 ? 0 : S.count;
      if (sel_mass) sel_mass[o] = S.sel_mass;
      if (sel_thresh) sel_thresh[o] = S.thr_key == 0u ? -INFINITY : okey_to_float(S.thr_key);
      if (sel_tie_last) sel_tie_last[o] = S.n_keys == 0 ? -1 : S.tie_last;
    }
  }
}

static int dbg_passes() {
  const char* e = getenv("RTP_DEBUG_MAX_PASSES");
  return e ? atoi(e) : kMaxPasses;
}

template <int G>
cudaError_t launch_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                         const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride, int32_t* sel_count,
                         float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status,
                         cudaStream_t st) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(select_chunk_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemC);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  constexpr int BMP = kCRows / G;
  const int n_row_tiles = (int)((rows.R + BMP - 1) / BMP);
  dim3 grid(n_row_tiles, d.n_ih);
  select_chunk_kernel<G><<<grid, kCThreads, kSmemC, st>>>(cv, d, hm, qt, rows.seq_id, rows.q_start, (int)rows.R,
                                                          sel_idx, sel_stride, sel_count, sel_mass, sel_thresh,
                                                          sel_tie_last, status, n_row_tiles, dbg_passes());
  return cudaGetLastError();
}

}  // namespace

size_t select_chunk_workspace_bytes(const Dims& d, int64_t R) {
  (void)d;
  (void)R;
  return 256;   // all state lives in shared memory
}

cudaError_t launch_select_chunk(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride,
                                int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  (void)ws;
  (void)sm_count;
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  int max_nh = 0;
  for (int j = 0; j < d.n_ih; ++j) max_nh = hm.ih_nheads[j] > max_nh ? hm.ih_nheads[j] : max_nh;
  // rows of a CTA are [head slot][position]: pick the smallest supported slot count that fits
  if (max_nh <= 1) return launch_typed<1>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, st);
  if (max_nh <= 2) return launch_typed<2>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, st);
  if (max_nh <= 4) return launch_typed<4>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, st);
  if (max_nh <= 8) return launch_typed<8>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, st);
  return cudaErrorNotSupported;
}

}  // namespace rtp
