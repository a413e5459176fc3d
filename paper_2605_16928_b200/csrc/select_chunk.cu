// S2-S4 for a prefill chunk: fused indexer + top-p selection (Eq. 5) for rows q_start .. q_start+C-1
// of one sequence.
//
// A CTA owns 128 (row, head) pairs: (128 / G) consecutive positions x the G retrieval heads of one
// index head; each warp owns 16 of them (one head, 16 positions).  The CTA streams the index keys
// 0 .. last position (2 KB per page, cp.async double buffer) once per pass; a warp scores a 64-key
// page against its 16 rows with eight m16n8k16 MMAs.  All selection state lives in shared memory, so
// the whole selection of the chunk is one kernel without inter-CTA communication:
//   max       row maximum M                                                   (1 op per score)
//   level 1   64-bin histogram of softmax mass over d = M - s in steps of 1/2 (d >= 31.25 pooled), in
//             fixed point with native 32-bit shared-memory adds; gives Z and the bucket in which the
//             cumulative mass reaches p * Z; the bucket becomes an exact interval of ordered score keys
//             (bisection) and of unscaled MMA outputs (so later passes compare raw values only)
//   key level 64-bin mass histogram of the ordered key inside the interval, 6 key bits per pass, until the
//             chosen bin provably holds at most 64 keys.  From here on only a small share of the scores falls
//             into a row's interval: a warp appends those hits (row, position, raw score) to a queue in shared
//             memory and works them off 32 at a time, one hit per lane, so that the per-hit arithmetic and the
//             shared-memory adds are issued once per 32 hits instead of once per MMA
//   collect   the keys of the final bucket go to a 64-entry list, the keys above it are counted; the warp
//             ranks the list exactly by (score descending, position ascending) and cuts it
//   tie       only when more than 64 equal scores straddle the cut: position of the last tie taken
// Rows drop out as soon as they are resolved; the CTA stops when all its rows are.  When id lists
// are requested, one more sweep appends every row's members in position order.
// Each pass has its own inner loop; pages that lie wholly below a warp's first row need no causal test.
#include <cstdlib>
#include "mass_hist.cuh"

namespace rtp {

namespace {

constexpr int kCWarps = 8;
constexpr int kCThreads = kCWarps * 32;
constexpr int kCRows = 128;
constexpr int kPagesPerStage = 4;
constexpr int kStageKeys = kPagesPerStage * kPage;                  // 256 keys
constexpr int kStageBytesC = kStageKeys * kIndexDim * 2;            // 8 KB
constexpr int kCandCapC = 64;                                       // candidates ranked exactly per row
constexpr int kCandCapG = 4096;                                     // candidates collected per row (global scratch), narrowed to kCandCapC in the warp
constexpr int kRowBytes = kBins * 8 + 8;                            // per row: 64 x {sum, carries} or 64 x {key, idx}; +8 staggers the banks
constexpr int kMaxPasses = 14;
constexpr float kLog2eC = kLog2eH;
constexpr int kQueueCap = 288;                                      // per-warp queue of bucket hits (entries of 8 bytes)

enum Phase { kPhMax = 0, kPhL1 = 1, kPhKey = 2, kPhCollect = 3, kPhTie = 4, kPhDone = 5 };

struct RowState {      // one per (row, head), in shared memory
  float M, Z, target, mass_above;
  float ref_s;         // key levels: masses are accumulated relative to exp(ref_s - M) (upper end of the level-1 bucket)
  float e_ref;         // exp(ref_s - M)
  uint32_t base_key;   // bucket = keys in [base_key, base_key + span)
  uint32_t span;
  int32_t shift;       // key levels: bin = (key - base_key) >> shift, in [0, 64)
  float raw_lo, raw_hi;   // unscaled-score interval of the bucket
  int32_t phase;
  int32_t cnt_above;   // keys strictly above the final bucket (counted in the collect pass)
  int32_t cand_cnt;    // keys inside the final bucket (collect pass)
  int32_t tie_need;    // tie pass: number of ties to take
  uint32_t thr_key;    // result: selected <=> key > thr_key or (key == thr_key and n <= tie_last)
  int32_t tie_last;
  int32_t n_keys;
  float sel_mass;
  int32_t count;
};

constexpr int kHistBytes = kCRows * kRowBytes;                      // 64 KB
constexpr int kQueueBytes = kCWarps * kQueueCap * 8;               // 18 KB
constexpr int kSmemC = kHistBytes + 2 * kStageBytesC + kQueueBytes + kCRows * (int)sizeof(RowState);

__device__ __forceinline__ void cp_async16c(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ uint32_t smem_u32c(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Per-lane view of its two rows for one pass (registers).
struct LaneRows {
  float M_a, M_b;
  int pos_a, pos_b;
  // Unscaled MMA outputs are compared directly: the keys of a bucket are the images of one closed interval of
  // raw values (finish_score is monotone), found by bisection when the bucket is chosen.
  float lo_a, hi_a, lo_b, hi_b;      // raw interval of the current bucket (empty: lo = +inf, hi = -inf)
  float mid_a, hw_a, mid_b, hw_b;    // the same interval as centre and half width (slightly widened): 2-op reject
  float cut_a, cut_b;                // collect pass: raw values above this are counted as above the bucket (+inf: none)
  float tlo_a, thi_a, tlo_b, thi_b;  // tie pass: raw interval of the tied key value
  float ref_a, ref_b;                // key levels: mass reference score
  uint32_t base_a, base_b;
  int shift_a, shift_b;
  bool collect_a, collect_b;         // the bucket's keys are collected instead of histogrammed
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
                                        const LaneRows& L, float scale, uint32_t* hist_a, uint32_t* hist_b) {
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
      const float s = s4[e] * scale;   // (the sign of a zero score does not matter here)
      const float M = lo ? L.M_a : L.M_b;
      float bin_f;
      const int bin = l1_bin_f(M, s, bin_f);   // (rows that are already done have no M: they land in bin 0)
      // mass relative to the bin's upper end: exp(-((M - s) - (bin/2 - 1/4))), scaled by 2^20
      add_mass((lo ? hist_a : hist_b) + 2 * bin, l1_mass_arg(M, s, bin_f));
    }
  }
}

// Key levels, candidate collection and (when TIE) the in-order tie count.  Rows that take no part carry empty
// intervals, so no per-row branching is needed on the common path.
template <bool MASK, bool TIE, bool COUNT>
__device__ __forceinline__ void page_late(const unsigned char* pg, const QFrag& iq, int lane, int n_page,
                                          const LaneRows& L, float scale, uint32_t* hist_a, uint32_t* hist_b,
                                          int* ccnt_a, int* ccnt_b, uint2* gc_a, uint2* gc_b, int& cnt_a, int& cnt_b,
                                          int need_a, int need_b, int& run_a, int& run_b, int& tl_a, int& tl_b) {
  const int g = lane >> 2, c = lane & 3;
  const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    const uint2 b = *reinterpret_cast<const uint2*>(pg + (nt * 8 + g) * (kIndexDim * 2) + boff);
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
    float s4[4];
    mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
    const int n0 = n_page + nt * 8 + 2 * c;
    if (MASK) {
      const float nan = __int_as_float(0x7fc00000);   // fails every test below
      if (n0 > L.pos_a) s4[0] = nan;
      if (n0 + 1 > L.pos_a) s4[1] = nan;
      if (n0 > L.pos_b) s4[2] = nan;
      if (n0 + 1 > L.pos_b) s4[3] = nan;
    }
    if (COUNT) {   // keys above the bucket of a row that is collecting
      cnt_a += (s4[0] > L.cut_a) + (s4[1] > L.cut_a);
      cnt_b += (s4[2] > L.cut_b) + (s4[3] > L.cut_b);
    }
    // quick reject: |raw - mid| <= hw is implied by raw in [lo, hi]
    const bool near = fabsf(s4[0] - L.mid_a) <= L.hw_a || fabsf(s4[1] - L.mid_a) <= L.hw_a ||
                      fabsf(s4[2] - L.mid_b) <= L.hw_b || fabsf(s4[3] - L.mid_b) <= L.hw_b;
    int tf_a = 0, tf_b = 0;
    if (near) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool lo = e < 2;
        const float raw = s4[e];
        if (raw >= (lo ? L.lo_a : L.lo_b) && raw <= (lo ? L.hi_a : L.hi_b)) {
          if (TIE && (lo ? L.tlo_a : L.tlo_b) <= raw && raw <= (lo ? L.thi_a : L.thi_b)) {
            if (lo) tf_a |= 1 << (e & 1); else tf_b |= 1 << (e & 1);
            continue;
          }
          const float s = finish_score(raw, scale);
          const uint32_t key = okey(s);
          uint32_t* h = lo ? hist_a : hist_b;
          if (lo ? L.collect_a : L.collect_b) {
            const int slot = atomicAdd(lo ? ccnt_a : ccnt_b, 1);
            if (slot < kCandCapG) (lo ? gc_a : gc_b)[slot] = make_uint2(key, (uint32_t)(n0 + (e & 1)));
          } else {
            const uint32_t t = key - (lo ? L.base_a : L.base_b);
            add_mass(h + 2 * (t >> (lo ? L.shift_a : L.shift_b)), fmaf(s - (lo ? L.ref_a : L.ref_b), kLog2eC, 20.0f));
          }
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

// Works off the warp's queue of bucket hits: entry = {position | local row << 27, raw score bits}.
// (The count is passed by value: a reference would pin the caller's counter to local memory.)
__device__ __noinline__ void drain_hits(uint32_t* wq, int qcnt, int lane, int wrow, RowState* rs, uint32_t* hist,
                                        uint2* gcand, float scale) {
  constexpr int kRowWords = kRowBytes / 4;
  __syncwarp();
  for (int base = 0; base < qcnt; base += 32) {
    const int i = base + lane;
    if (i < qcnt) {
      const uint32_t w0 = wq[2 * i];
      const float raw = __uint_as_float(wq[2 * i + 1]);
      const int r = wrow + (int)(w0 >> 27);
      RowState* S = rs + r;
      const float s = finish_score(raw, scale);
      const uint32_t key = okey(s);
      uint32_t* h = hist + r * kRowWords;
      if (S->phase == kPhCollect) {
        const int slot = atomicAdd(&S->cand_cnt, 1);
        if (slot < kCandCapG) gcand[(size_t)r * kCandCapG + slot] = make_uint2(key, w0 & 0x7ffffffu);
      } else {
        const uint32_t t = key - S->base_key;
        add_mass(h + 2 * (t >> S->shift), fmaf(s - S->ref_s, kLog2eC, 20.0f));
      }
    }
  }
  __syncwarp();
}

// Key levels and candidate collection without ties: hits go to the warp's queue.
template <bool MASK, bool COUNT>
__device__ __forceinline__ void page_hits(const unsigned char* pg, const QFrag& iq, int lane, int n_page,
                                          const LaneRows& L, int& cnt_a, int& cnt_b, uint32_t* wq, int& qcnt,
                                          int wrow, RowState* rs, uint32_t* hist, uint2* gcand, float scale) {
  const int g = lane >> 2, c = lane & 3;
  const int boff = 2 * qfrag_dim_offset(lane);
  // Four 8-key groups at a time: their MMAs and interval tests are issued back to back, and one vote decides whether
  // any of the 512 scores is a hit (the usual answer in the later passes is no).
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    float s[4][4];
    uint32_t hits = 0;   // bit 4 q + e: score e of group q is inside its row's bucket
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int nt = half * 4 + q;
      const uint2 b = *reinterpret_cast<const uint2*>(pg + (nt * 8 + g) * (kIndexDim * 2) + boff);
      const float zero[4] = {0.f, 0.f, 0.f, 0.f};
      mma_bf16_16816(s[q], iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int n0 = n_page + (half * 4 + q) * 8 + 2 * c;
      if (MASK) {
        const float nan = __int_as_float(0x7fc00000);   // fails every test below
        if (n0 > L.pos_a) s[q][0] = nan;
        if (n0 + 1 > L.pos_a) s[q][1] = nan;
        if (n0 > L.pos_b) s[q][2] = nan;
        if (n0 + 1 > L.pos_b) s[q][3] = nan;
      }
      if (COUNT) {   // keys above the bucket of a row that is collecting
        cnt_a += (s[q][0] > L.cut_a) + (s[q][1] > L.cut_a);
        cnt_b += (s[q][2] > L.cut_b) + (s[q][3] > L.cut_b);
      }
      if (s[q][0] >= L.lo_a && s[q][0] <= L.hi_a) hits |= 1u << (4 * q);
      if (s[q][1] >= L.lo_a && s[q][1] <= L.hi_a) hits |= 2u << (4 * q);
      if (s[q][2] >= L.lo_b && s[q][2] <= L.hi_b) hits |= 4u << (4 * q);
      if (s[q][3] >= L.lo_b && s[q][3] <= L.hi_b) hits |= 8u << (4 * q);
    }
    if (!__any_sync(0xffffffffu, hits != 0u)) continue;
    // every lane appends its hits behind those of the lower lanes: a prefix sum over the lanes' hit counts, then
    // predicated stores (no vote per score); two 8-key groups at a time bound the queue growth by 256 entries
#pragma unroll
    for (int pr = 0; pr < 2; ++pr) {
      const uint32_t hb = (hits >> (8 * pr)) & 0xffu;
      const int mine = __popc(hb);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      int pos = qcnt + incl - mine;
      qcnt += __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
      for (int qq = 0; qq < 2; ++qq) {
        const int q = 2 * pr + qq;
        const int n0 = n_page + (half * 4 + q) * 8 + 2 * c;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if ((hb >> (4 * qq + e)) & 1u) {
            wq[2 * pos] = (uint32_t)(n0 + (e & 1)) | ((uint32_t)(g + (e >> 1) * 8) << 27);
            wq[2 * pos + 1] = __float_as_uint(s[q][e]);
            ++pos;
          }
        }
      }
      if (qcnt >= 32) {   // at most 31 + 256 entries queued
        drain_hits(wq, qcnt, lane, wrow, rs, hist, gcand, scale);
        qcnt = 0;
      }
    }
  }
}

template <int G>
__global__ void __launch_bounds__(kCThreads, 2) select_chunk_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const __nv_bfloat16* __restrict__ qt,
    const int seq_id, const int q_start, const int C, int32_t* __restrict__ sel_idx, const int64_t sel_stride,
    int32_t* __restrict__ sel_count, float* __restrict__ sel_mass, float* __restrict__ sel_thresh,
    int32_t* __restrict__ sel_tie_last, int32_t* status, uint2* __restrict__ gcand_all, const int n_row_tiles,
    const int max_passes) {
  constexpr int BMP = kCRows / G;
  // candidate scratch of this CTA: [128 rows][kCandCapG] {ordered key, position}
  uint2* gcand = gcand_all + ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * (size_t)(kCRows * kCandCapG);
  extern __shared__ __align__(128) unsigned char smem[];
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem);                      // [128 rows][128 words]
  unsigned char* stage_s = smem + kHistBytes;
  uint32_t* queue = reinterpret_cast<uint32_t*>(smem + kHistBytes + 2 * kStageBytesC);
  RowState* rs = reinterpret_cast<RowState*>(smem + kHistBytes + 2 * kStageBytesC + kQueueBytes);
  __shared__ int s_pending;
  constexpr int kRowWords = kRowBytes / 4;

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
  uint32_t* hist_a = hist + la * kRowWords;
  uint32_t* hist_b = hist + lb * kRowWords;
  const float scale = d.score_scale;
  const float kInf = __int_as_float(0x7f800000);

  for (int pass = 0; pass < max_passes; ++pass) {
    // ---- what does this pass do for my two rows? ----
    const RowState sa = rs[la], sb = rs[lb];
    const int ph_a = a_ok ? sa.phase : kPhDone, ph_b = b_ok ? sb.phase : kPhDone;
    if (tid == 0) s_pending = 0;
    for (int i = lane; i < 16 * kRowWords; i += 32) hist[wrow * kRowWords + i] = 0u;   // this warp's rows
    __syncthreads();
    const bool warp_active = __any_sync(0xffffffffu, ph_a != kPhDone || ph_b != kPhDone);
    // All rows of a warp do the max pass and the level-1 pass together; later passes mix key levels,
    // candidate collection and ties.
    const bool pass_max = __any_sync(0xffffffffu, ph_a == kPhMax || ph_b == kPhMax);
    const bool pass_l1 = __any_sync(0xffffffffu, ph_a == kPhL1 || ph_b == kPhL1);
    const bool pass_tie = __any_sync(0xffffffffu, ph_a == kPhTie || ph_b == kPhTie);
    const bool pass_count = __any_sync(0xffffffffu, ph_a == kPhCollect || ph_b == kPhCollect);

    LaneRows LR;
    LR.M_a = sa.M; LR.M_b = sb.M;
    LR.pos_a = pos_a; LR.pos_b = pos_b;
    LR.base_a = sa.base_key; LR.base_b = sb.base_key;
    LR.shift_a = sa.shift; LR.shift_b = sb.shift;
    LR.ref_a = sa.ref_s; LR.ref_b = sb.ref_s;
    const bool in_a = ph_a == kPhKey || ph_a == kPhCollect || ph_a == kPhTie;
    const bool in_b = ph_b == kPhKey || ph_b == kPhCollect || ph_b == kPhTie;
    LR.lo_a = in_a ? sa.raw_lo : kInf;  LR.hi_a = in_a ? sa.raw_hi : -kInf;
    LR.lo_b = in_b ? sb.raw_lo : kInf;  LR.hi_b = in_b ? sb.raw_hi : -kInf;
    // centre / half width of the interval; the half width is rounded up so that the quick test never rejects a member
    LR.mid_a = in_a ? 0.5f * sa.raw_lo + 0.5f * sa.raw_hi : 0.f;
    LR.mid_b = in_b ? 0.5f * sb.raw_lo + 0.5f * sb.raw_hi : 0.f;
    LR.hw_a = in_a ? fmaxf(sa.raw_hi - LR.mid_a, LR.mid_a - sa.raw_lo) * 1.000001f + 1e-30f : -1.f;
    LR.hw_b = in_b ? fmaxf(sb.raw_hi - LR.mid_b, LR.mid_b - sb.raw_lo) * 1.000001f + 1e-30f : -1.f;
    LR.collect_a = ph_a == kPhCollect;  LR.collect_b = ph_b == kPhCollect;
    LR.cut_a = LR.collect_a ? sa.raw_hi : kInf;
    LR.cut_b = LR.collect_b ? sb.raw_hi : kInf;
    const bool tie_a = ph_a == kPhTie, tie_b = ph_b == kPhTie;
    LR.tlo_a = tie_a ? sa.raw_lo : kInf;  LR.thi_a = tie_a ? sa.raw_hi : -kInf;
    LR.tlo_b = tie_b ? sb.raw_lo : kInf;  LR.thi_b = tie_b ? sb.raw_hi : -kInf;
    const int need_a = tie_a ? sa.tie_need : 0, need_b = tie_b ? sb.tie_need : 0;
    int* ccnt_a = &rs[la].cand_cnt;
    int* ccnt_b = &rs[lb].cand_cnt;

    float mx_a = -INFINITY, mx_b = -INFINITY;
    int cnt_a = 0, cnt_b = 0;
    int run_a = 0, run_b = 0;
    int tl_a = -1, tl_b = -1;
    uint32_t* wq = queue + warp * (kQueueCap * 2);
    int qcnt = 0;

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
          } else {
#define RTP_LATE(M_, T_, C_) page_late<M_, T_, C_>(pgp, iq, lane, n_page, LR, scale, hist_a, hist_b, ccnt_a, ccnt_b, gcand + (size_t)la * kCandCapG, gcand + (size_t)lb * kCandCapG, cnt_a, cnt_b, need_a, need_b, run_a, run_b, tl_a, tl_b)
#define RTP_HITS(M_, C_) page_hits<M_, C_>(pgp, iq, lane, n_page, LR, cnt_a, cnt_b, wq, qcnt, wrow, rs, hist, gcand, scale)
            if (pass_tie) {
              if (interior) RTP_LATE(false, true, true); else RTP_LATE(true, true, true);
            } else if (pass_count) {
              if (interior) RTP_HITS(false, true); else RTP_HITS(true, true);
            } else {
              if (interior) RTP_HITS(false, false); else RTP_HITS(true, false);
            }
#undef RTP_LATE
#undef RTP_HITS
          }
        }
      }
      __syncthreads();
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (qcnt > 0) drain_hits(wq, qcnt, lane, wrow, rs, hist, gcand, scale);
    qcnt = 0;

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
      const uint32_t* h = hist + lr * kRowWords;
      if (ph == kPhDone || R.n_keys == 0) continue;
      if (ph == kPhMax) {
        // the maximum was taken on unscaled MMA outputs; scaling by a positive factor is monotone
        const float M = finish_score(__shfl_sync(0xffffffffu, is_b ? mx_b : mx_a, src_lane), scale);
        if (lane == 0) {
          S->M = M;
          S->phase = kPhL1;
        }
      } else if (ph == kPhL1 || ph == kPhKey) {
        // 64 bins of {hi, lo}; two bins per lane in order of decreasing score:
        //   level 1: bin 0 is the top -> lane l takes bins 2l, 2l+1;  key levels: bin 63 is the top -> 63-2l, 62-2l
        const bool l1 = ph == kPhL1;
        const int b0 = l1 ? 2 * lane : 63 - 2 * lane, b1 = l1 ? 2 * lane + 1 : 62 - 2 * lane;
        const uint32_t sum0 = h[2 * b0], car0 = h[2 * b0 + 1], sum1 = h[2 * b1], car1 = h[2 * b1 + 1];
        const float q0 = acc_mass(sum0, car0), q1 = acc_mass(sum1, car1);
        // masses relative to M
        float m0f, m1f;
        if (l1) {
          m0f = q0 * l1_bin_scale(b0);
          m1f = q1 * l1_bin_scale(b1);
        } else {
          const float sc = R.e_ref * 9.5367431640625e-07f;   // 2^-20
          m0f = q0 * sc;
          m1f = q1 * sc;
        }
        float incm = m0f + m1f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float tm = __shfl_up_sync(0xffffffffu, incm, o);
          if (lane >= o) incm += tm;
        }
        const float total = __shfl_sync(0xffffffffu, incm, 31);
        const float Z = l1 ? total : R.Z;
        const float target = l1 ? d.top_p * Z * (1.0f + kMassMargin) : R.target;
        const float run = (l1 ? 0.f : R.mass_above) + incm - (m0f + m1f);
        const bool pop0 = (sum0 | car0) != 0u, pop1 = (sum1 | car1) != 0u;
        // order index of a bin = position from the top (0 .. 63)
        int found = 64, last = -1;
        if (pop0) {
          last = 2 * lane;
          if (run + m0f >= target) found = 2 * lane;
        }
        if (pop1) {
          last = 2 * lane + 1;
          if (found == 64 && run + m0f + m1f >= target) found = 2 * lane + 1;
        }
        int best = found;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
        if (best == 64) best = last;   // rounding left the target just out of reach: lowest populated bin
        if (best < 0) {
          if (lane == 0) {             // empty histogram: cannot happen for a non-empty row
            S->phase = kPhDone;
            set_status(status, RTP_ERR_UNSUPPORTED);
          }
        } else if ((best >> 1) == lane) {
          const bool first = (best & 1) == 0;
          const float f_above = first ? run : run + m0f;
          const float f_q = first ? q0 : q1;
          const int bin = first ? b0 : b1;
          const bool few = f_q < 0.999f * kMinQ * (float)kCandCapG;   // fewer than kCandCapG keys in the bin
          S->mass_above = f_above;
          if (l1) {
            S->Z = Z;
            S->target = target;
            if (bin == kBins - 1) {
              // the cut falls into the pooled tail (mass below 2e-14 per key): take every key
              S->thr_key = 0u;
              S->tie_last = R.n_keys - 1;
              S->count = R.n_keys;
              S->sel_mass = 1.0f;
              S->phase = kPhDone;
            } else {
              const float M = R.M;
              const float hi_s = l1_bin_hi(M, bin);
              uint32_t klo, khi;
              l1_bin_keys(M, bin, klo, khi);
              const uint32_t span = khi - klo + 1u;
              const int bits = span > 1u ? 32 - __clz(span - 1u) : 0;
              float rlo, rhi;
              raw_preimage(scale, klo, khi, rlo, rhi);
              S->ref_s = hi_s;
              S->e_ref = fast_ex2(-kLog2eC * (0.5f * (float)bin - 0.25f));
              S->base_key = klo;
              S->span = span;
              S->shift = max(0, bits - 6);
              S->raw_lo = rlo;
              S->raw_hi = rhi;
              S->cand_cnt = 0;
              S->phase = (few || span == 1u) ? kPhCollect : kPhKey;
            }
          } else {
            const int shift = R.shift;
            const uint32_t ofs = (uint32_t)bin << shift;
            const uint32_t lo_key = R.base_key + ofs;
            const uint32_t sub_span = min(1u << shift, R.span - ofs);
            float rlo, rhi;
            raw_preimage(scale, lo_key, lo_key + (sub_span - 1u), rlo, rhi);
            S->base_key = lo_key;
            S->span = sub_span;
            S->shift = max(0, shift - 6);
            S->raw_lo = rlo;
            S->raw_hi = rhi;
            S->cand_cnt = 0;
            S->phase = (few || sub_span == 1u) ? kPhCollect : kPhKey;
          }
        }
      } else if (ph == kPhCollect) {
        // The pass put every key of the bucket (at most kCandCapG, by the bound that sent the row here) into the row's
        // list in global scratch and counted the keys above the bucket.  While more than kCandCapC of them are left,
        // the warp narrows on the list itself: the same 64-bin mass histogram over the next six key bits, in the row's
        // shared-memory bins, no pass over the keys.  Then the exact ranking below finishes.
        const int n_all = R.cand_cnt;
        int above = R.cnt_above + __shfl_sync(0xffffffffu, is_b ? cnt_b : cnt_a, src_lane);
        float m_above = R.mass_above;
        uint32_t base = R.base_key, span = R.span;
        int n_in = n_all;
        const uint2* gc = gcand + (size_t)lr * kCandCapG;
        uint32_t* hw = hist + lr * kRowWords;
        if (n_all <= kCandCapG) {
          while (n_in > kCandCapC && span > 1u) {
            const int bits = 32 - __clz(span - 1u);
            const int shift = max(0, bits - 6);
            for (int i = lane; i < kRowWords; i += 32) hw[i] = 0u;
            __syncwarp();
            for (int i = lane; i < n_all; i += 32) {
              const uint32_t key = __ldcg(&gc[i].x);
              const uint32_t t = key - base;
              if (t < span) add_mass(hw + 2 * (t >> shift), fmaf(okey_to_float(key) - R.ref_s, kLog2eC, 20.0f));
            }
            __syncwarp();
            const int b0 = 63 - 2 * lane, b1 = 62 - 2 * lane;   // bin 63 is the top
            const uint32_t sum0 = hw[2 * b0], car0 = hw[2 * b0 + 1], sum1 = hw[2 * b1], car1 = hw[2 * b1 + 1];
            const float sc = R.e_ref * 9.5367431640625e-07f;     // 2^-20
            const float m0f = acc_mass(sum0, car0) * sc, m1f = acc_mass(sum1, car1) * sc;
            float incm = m0f + m1f;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const float tm = __shfl_up_sync(0xffffffffu, incm, o);
              if (lane >= o) incm += tm;
            }
            const float run = m_above + incm - (m0f + m1f);
            int found = 64, last = -1;
            if (sum0 | car0) {
              last = 2 * lane;
              if (run + m0f >= R.target) found = 2 * lane;
            }
            if (sum1 | car1) {
              last = 2 * lane + 1;
              if (found == 64 && run + m0f + m1f >= R.target) found = 2 * lane + 1;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
              last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
            }
            if (found == 64) found = last;
            if (found < 0) break;                                 // (no candidate inside the interval: cannot happen)
            m_above = __shfl_sync(0xffffffffu, (found & 1) ? run + m0f : run, found >> 1);
            const uint32_t ofs = (uint32_t)(63 - found) << shift;
            const uint32_t nbase = base + ofs, nspan = min(1u << shift, span - ofs);
            int c_in = 0, c_up = 0;                               // candidates inside / above the new interval
            for (int i = lane; i < n_all; i += 32) {
              const uint32_t t = __ldcg(&gc[i].x) - base;
              if (t < span) {
                if (t - ofs < nspan) ++c_in;
                else if (t >= ofs) ++c_up;
              }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              c_in += __shfl_xor_sync(0xffffffffu, c_in, o);
              c_up += __shfl_xor_sync(0xffffffffu, c_up, o);
            }
            above += c_up;
            n_in = c_in;
            base = nbase;
            span = nspan;
            __syncwarp();
          }
        }
        if (n_in > kCandCapC) {
          // more than kCandCapC keys share one key value: n_in equal scores straddle the cut
          float rlo = 0.f, rhi = 0.f;
          if (lane == 0 && base != R.base_key) raw_preimage(scale, base, base, rlo, rhi);
          if (lane == 0) {
            const float each = fast_ex2((okey_to_float(base) - R.M) * kLog2eC);
            int take = (int)ceilf((R.target - m_above) / each);
            take = max(1, min(take, n_in));
            S->cnt_above = above;
            S->mass_above = m_above;
            S->thr_key = base;
            S->count = above + take;
            S->sel_mass = (m_above + (float)take * each) / R.Z;
            if (span != 1u) set_status(status, RTP_ERR_UNSUPPORTED);
            if (take < n_in) {
              if (base != R.base_key) {   // the tie pass looks for this key value
                S->base_key = base;
                S->span = 1u;
                S->raw_lo = rlo;
                S->raw_hi = rhi;
              }
              S->tie_need = take;
              S->phase = kPhTie;
            } else {
              S->tie_last = R.n_keys - 1;
              S->phase = kPhDone;
            }
          }
        } else {
          // the candidates of the final interval move into the row's shared-memory list {key, position}
          __syncwarp();
          int filled = 0;
          for (int i0 = 0; i0 < n_all; i0 += 32) {
            const int i = i0 + lane;
            uint2 cnd = make_uint2(0u, 0u);
            bool in = false;
            if (i < n_all) {
              cnd = __ldcg(&gc[i]);
              in = cnd.x - base < span;
            }
            const uint32_t m = __ballot_sync(0xffffffffu, in);
            if (in) {
              const int pos = filled + __popc(m & ((1u << lane) - 1u));
              hw[2 * pos] = cnd.x;
              hw[2 * pos + 1] = cnd.y;
            }
            filled += __popc(m);
          }
          __syncwarp();
          const int n_c = n_in;
          // exact finish: rank the (at most 64) candidates by (score descending, position ascending)
          unsigned long long ord[2];
          float e[2];
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int i = 2 * lane + x;
            ord[x] = ~0ull;
            e[x] = 0.f;
            if (i < n_c) {
              const uint32_t key = h[2 * i], idx = h[2 * i + 1];
              ord[x] = ((unsigned long long)(~key) << 32) | idx;
              e[x] = fast_ex2((okey_to_float(key) - R.M) * kLog2eC);
            }
          }
          int rank[2] = {0, 0};
          float cum[2] = {m_above, m_above};
          for (int j = 0; j < n_c; ++j) {
            const int jl = j >> 1;
            const unsigned long long oj = __shfl_sync(0xffffffffu, (j & 1) ? ord[1] : ord[0], jl);
            const float ej = __shfl_sync(0xffffffffu, (j & 1) ? e[1] : e[0], jl);
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              if (oj < ord[x]) ++rank[x];
              if (oj <= ord[x]) cum[x] += ej;
            }
          }
          // shortest prefix whose cumulative mass reaches the target (all candidates if none does)
          int pick = 1 << 20;
#pragma unroll
          for (int x = 0; x < 2; ++x)
            if (2 * lane + x < n_c && cum[x] >= R.target) pick = min(pick, rank[x]);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) pick = min(pick, __shfl_xor_sync(0xffffffffu, pick, o));
          if (pick == (1 << 20)) pick = n_c - 1;
          // the candidate of rank `pick` defines the threshold; ties with it that were taken have rank <= pick
          uint32_t thr_key = 0;
          float pick_cum = 0.f;
#pragma unroll
          for (int x = 0; x < 2; ++x)
            if (2 * lane + x < n_c && rank[x] == pick) {
              thr_key = ~(uint32_t)(ord[x] >> 32);
              pick_cum = cum[x];
            }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            thr_key = max(thr_key, __shfl_xor_sync(0xffffffffu, thr_key, o));
            pick_cum = fmaxf(pick_cum, __shfl_xor_sync(0xffffffffu, pick_cum, o));
          }
          // Position bound for keys that tie with the threshold score: the last one taken, or the row's last key
          // when none is left out (the usual case: then the attention kernel never has to look at positions).
          int tie_last = -1, left_out = 0;
#pragma unroll
          for (int x = 0; x < 2; ++x)
            if (2 * lane + x < n_c && ~(uint32_t)(ord[x] >> 32) == thr_key) {
              if (rank[x] <= pick) tie_last = max(tie_last, (int)(uint32_t)ord[x]); else left_out = 1;
            }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) tie_last = max(tie_last, __shfl_xor_sync(0xffffffffu, tie_last, o));
          if (!__any_sync(0xffffffffu, left_out)) tie_last = R.n_keys - 1;
          if (lane == 0) {
            S->cnt_above = above;
            S->thr_key = thr_key;
            S->tie_last = tie_last;
            S->count = above + pick + 1;
            S->sel_mass = pick_cum / R.Z;
            S->phase = kPhDone;
            if (n_c == 0) set_status(status, RTP_ERR_UNSUPPORTED);   // a chosen bucket always holds a key
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


template <int G>
cudaError_t launch_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                         const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride, int32_t* sel_count,
                         float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* ws,
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
                                                          sel_tie_last, status, reinterpret_cast<uint2*>(ws), n_row_tiles,
                                                          kMaxPasses);
  return cudaGetLastError();
}

}  // namespace

// rows of a CTA are [head slot][position]: the smallest supported slot count that fits the widest index head
static int slot_class(const Dims& d, const HeadMaps& hm) {
  int max_nh = 0;
  for (int j = 0; j < d.n_ih; ++j) max_nh = hm.ih_nheads[j] > max_nh ? hm.ih_nheads[j] : max_nh;
  return max_nh <= 1 ? 1 : max_nh <= 2 ? 2 : max_nh <= 4 ? 4 : max_nh <= 8 ? 8 : 0;
}

// Candidate scratch: kCandCapG entries of 8 bytes per (row, head slot) of every CTA.
size_t select_chunk_workspace_bytes(const Dims& d, const HeadMaps& hm, int64_t R) {
  const int g = slot_class(d, hm);
  if (g == 0 || R <= 0) return 256;
  const int64_t n_row_tiles = (R + kCRows / g - 1) / (kCRows / g);
  return (size_t)n_row_tiles * d.n_ih * kCRows * kCandCapG * sizeof(uint2);
}

cudaError_t launch_select_chunk(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride,
                                int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  (void)sm_count;
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  switch (slot_class(d, hm)) {
    case 1: return launch_typed<1>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, st);
    case 2: return launch_typed<2>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, st);
    case 4: return launch_typed<4>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, st);
    case 8: return launch_typed<8>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace rtp
