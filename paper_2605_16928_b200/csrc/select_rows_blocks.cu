// Block-wise top-p for explicit rows (the decode path), Section 3.4: the index keys of a row are cut into blocks of
// one cache page (64 keys), every block is reduced to a log-sum-exp pair (m_b, l_b), blocks are taken in order of
// decreasing m_b (equal maxima: smaller block first) until their softmax mass l_b exp(m_b - M) / Z reaches p.
//
//   blk_stats_kernel    one scan of the index keys: a warp scores a page for the unit's heads (MMA, see score16) and
//                       reduces it to (m_b, l_b) per head; nothing else is stored (8 bytes per head and page).
//   blk_select_kernel   one CTA per (row, head): block masses go into a 1024-bin histogram indexed by M - m_b (the
//                       paper's histogram indexed by m_b, finer and in exact integer arithmetic); the bins are scanned
//                       from the top until the mass reaches the target; blocks above the threshold's bin are selected,
//                       the blocks inside it are sorted by (m_b desc, block asc) in shared memory and the shortest
//                       prefix that completes the target is taken.  The result is a list of logical page numbers.
//
// The paper's kernel takes the threshold's bin whole; resolving the order inside it makes the selection the one the
// block-wise rule defines, not a superset of it.
#include "row_scan.cuh"

namespace rtp {

namespace {

using namespace rowscan;

constexpr float kLog2eB = 1.4426950408889634f;
constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxBlocksRow = 16384;   // blocks of a row the select kernel sorts in shared memory (1M keys)

// ---- pass 1: (m_b, l_b) of every page of the unit's slice ---------------------------------------------------------
// stats: float2 [rows * retrieval heads][nb_pad]; entry b = (largest finished score of block b, sum of exp(s - m_b)).
template <bool NH4, bool F8>
__global__ void __launch_bounds__(kThreads, NH4 ? 4 : 3) blk_stats_kernel(const CacheView cv, const Dims d, const HeadMaps hm,
                                                             const Rows rows, const __nv_bfloat16* __restrict__ qt,
                                                             float2* __restrict__ stats, const int64_t nb_pad,
                                                             int n_splits, int32_t* status) {
  chain_wait();
  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, status);
  if (x.p_lo >= x.p_hi) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  QFrag qf = load_qfrag(qt + x.r * d.n_ret * kIndexDim, hm.ih_heads[x.ih], x.nh, lane);
  if (F8 && !qfrag_to_f16(qf)) set_status(status, RTP_ERR_UNSUPPORTED);   // a projected query beyond fp16's range
  const int slot_a = elem_slot<NH4>(lane, 0), slot_b = NH4 ? slot_a : elem_slot<NH4>(lane, 4);
  float2* st_a = slot_a < x.nh ? stats + (x.r * d.n_ret + hm.ih_heads[x.ih][slot_a]) * nb_pad : nullptr;
  float2* st_b = (!NH4 && slot_b < x.nh) ? stats + (x.r * d.n_ret + hm.ih_heads[x.ih][slot_b]) * nb_pad : nullptr;
  // the lane of a head slot that writes the pair: NH4: (g < 4, c = 0); otherwise c = 0 (slots g and g + 8)
  const bool writer = NH4 ? ((lane & 3) == 0 && lane < 16) : ((lane & 3) == 0);
  constexpr int kN = LaneElems<NH4>::kN;
  uint4 v[4], vn[4];
  if (x.p_lo + warp < x.p_hi) load_page<F8>(cv, x, x.p_lo + warp, lane, vn);
  for (int p = x.p_lo + warp; p < x.p_hi; p += kWarps) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = vn[i];
    if (p + kWarps < x.p_hi) load_page<F8>(cv, x, p + kWarps, lane, vn);   // in flight while this page is worked on
    const bool tail = (p + 1) * kPage > x.n_keys;
    float fs[4][kN];
    float ma = -INFINITY, mb = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s_lo[4], s_hi[4];
      if (F8) score16_f8(qf, make_uint2(v[i].x, v[i].y), lane, s_lo, s_hi); else score16(qf, v[i], lane, s_lo, s_hi);
      const LaneElems<NH4> el = lane_elems<NH4>(s_lo, s_hi, lane);
#pragma unroll
      for (int e = 0; e < kN; ++e) {
        const bool beyond = tail && p * kPage + i * 16 + el.koff[e] >= x.n_keys;
        fs[i][e] = beyond ? -INFINITY : finish_score(el.raw[e], d.score_scale);
        if (NH4 || e < 4) ma = fmaxf(ma, fs[i][e]); else mb = fmaxf(mb, fs[i][e]);
      }
    }
    ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, 1));
    ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, 2));
    if (NH4) ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, 16));
    if (!NH4) {
      mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 1));
      mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 2));
    }
    // (a page of the slice holds at least one causal key, so ma and mb are finite for the slots in use)
    float la = 0.f, lb = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int e = 0; e < kN; ++e) {
        if (NH4 || e < 4) la += fast_ex2((fs[i][e] - ma) * kLog2eB); else lb += fast_ex2((fs[i][e] - mb) * kLog2eB);
      }
    }
    la += __shfl_xor_sync(0xffffffffu, la, 1);
    la += __shfl_xor_sync(0xffffffffu, la, 2);
    if (NH4) la += __shfl_xor_sync(0xffffffffu, la, 16);
    if (!NH4) {
      lb += __shfl_xor_sync(0xffffffffu, lb, 1);
      lb += __shfl_xor_sync(0xffffffffu, lb, 2);
    }
    if (writer) {
      if (st_a) st_a[p] = make_float2(ma, la);
      if (st_b) st_b[p] = make_float2(mb, lb);
    }
  }
}

// ---- pass 2: histogram over M - m_b, exact order inside the threshold's bin ---------------------------------------
// Dynamic shared memory: np2 sort keys of 8 bytes ((~ordered key of m_b) << 32 | block: ascending order = larger m_b
// first, then smaller block) followed by nb_pad floats (l_b by block number).
constexpr int kHistBins = 1024;           // bins of 1/32 in M - m_b: 32 units; everything deeper shares the last bin
constexpr float kHistScale = 32.0f;
// Block masses (at most 64 each, relative to exp(M)) are summed as integers at 2^24, so that the sums do not depend on
// the order of the adds: a bin is {sum mod 2^32, carries}, added to with native 32-bit shared-memory atomics.
constexpr float kFix = 16777216.0f;

__global__ void __launch_bounds__(kSelThreads) blk_select_kernel(
    const CacheView cv, const Dims d, const Rows rows, const float2* __restrict__ stats, const int64_t nb_pad,
    const int np2, int32_t* __restrict__ blk_idx, const int64_t blk_stride, int32_t* __restrict__ sel_count,
    float* __restrict__ sel_mass, float* __restrict__ sel_thresh, int32_t* __restrict__ sel_tie_last, int32_t* status) {
  chain_wait();
  extern __shared__ __align__(16) unsigned char blk_smem[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(blk_smem);
  float* lw = reinterpret_cast<float*>(blk_smem + (size_t)np2 * 8);
  __shared__ uint32_t hist2[kHistBins][2];
  auto hist_at = [&](int b) -> unsigned long long { return ((unsigned long long)hist2[b][1] << 32) | hist2[b][0]; };
  __shared__ unsigned long long w_tot[kSelWarps];
  __shared__ float w_sum[kSelWarps];
  __shared__ uint32_t w_max[kSelWarps];
  __shared__ int s_pick, s_bin, s_n_in, s_n_above;
  __shared__ unsigned long long s_above;
  __shared__ float s_run, s_pick_mass;
  const int64_t rh = blockIdx.x;
  const int64_t r = rh / d.n_ret;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seq = rows.row_seq(r);
  int n_keys = rows.row_pos(r) + 1;
  {
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;
    n_keys = max(0, min(n_keys, sl));
  }
  const int nb = (n_keys + kPage - 1) >> kPageShift;
  int32_t* out_ids = blk_idx ? blk_idx + rh * blk_stride : nullptr;
  if (nb == 0) {
    if (tid == 0) {
      sel_count[rh] = 0;
      if (sel_mass) sel_mass[rh] = 0.f;
      if (sel_thresh) sel_thresh[rh] = 0.f;
      if (sel_tie_last) sel_tie_last[rh] = -1;
    }
    return;
  }
  const float2* st = stats + rh * nb_pad;
  if (d.top_p >= 1.0f || nb <= 1) {   // every block
    if (out_ids)
      for (int i = tid; i < nb; i += kSelThreads)
        if (i < blk_stride) out_ids[i] = i;
    if (tid == 0) {
      sel_count[rh] = nb;
      if (sel_mass) sel_mass[rh] = 1.0f;
      if (sel_thresh) sel_thresh[rh] = -INFINITY;
      if (sel_tie_last) sel_tie_last[rh] = nb - 1;
      if (out_ids && nb > blk_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }
  // A thread keeps the pairs of its (at most 16) blocks in registers: all loads are in flight together.  M, and the
  // l_b by block number for the ordered scan at the end.
  constexpr int kMine = kMaxBlocksRow / kSelThreads;
  float m_r[kMine], l_r[kMine];
  uint32_t kmax = 0u;
#pragma unroll
  for (int k = 0; k < kMine; ++k) {
    const int i = tid + k * kSelThreads;
    float2 s = make_float2(-INFINITY, 0.f);
    if (i < nb) s = __ldcg(st + i);
    m_r[k] = s.x;
    l_r[k] = s.y;
  }
#pragma unroll
  for (int k = 0; k < kMine; ++k) {
    const int i = tid + k * kSelThreads;
    if (i < nb) {
      kmax = max(kmax, okey(m_r[k]));
      lw[i] = l_r[k];
    }
  }
  for (int i = tid; i < 2 * kHistBins; i += kSelThreads) (&hist2[0][0])[i] = 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  if (lane == 0) w_max[warp] = kmax;
  if (tid == 0) {
    s_pick = 0x7fffffff;
    s_run = 0.f;
    s_pick_mass = 0.f;
    s_n_in = 0;
    s_n_above = 0;
  }
  __syncthreads();
  for (int w = 0; w < kSelWarps; ++w) kmax = max(kmax, w_max[w]);
  const float M = okey_to_float(kmax);
  auto bin_of = [&](float m) -> int { return (int)fminf((M - m) * kHistScale, (float)(kHistBins - 1)); };   // monotone in m
  auto mass_of = [&](float m, float l) -> float { return l * fast_ex2((m - M) * kLog2eB); };                 // relative to exp(M)
  // histogram of block masses, integers: the sums do not depend on the order of the adds
  unsigned long long mine = 0ull;
#pragma unroll
  for (int k = 0; k < kMine; ++k) {
    if (tid + k * kSelThreads >= nb) continue;
    const uint32_t q = (uint32_t)(mass_of(m_r[k], l_r[k]) * kFix);   // (below 2^31)
    uint32_t* acc = hist2[bin_of(m_r[k])];
    const uint32_t old = atomicAdd(acc, q);
    if (old + q < old) atomicAdd(acc + 1, 1u);
    mine += q;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
  if (lane == 0) w_tot[warp] = mine;
  __syncthreads();
  unsigned long long Zq = 0ull;
  for (int w = 0; w < kSelWarps; ++w) Zq += w_tot[w];
  const float Z = (float)Zq / kFix;
  const float target = d.top_p * Z * (1.0f + kMassMargin);
  // the threshold's bin: the first from the top at which the cumulative mass reaches the target (warp 0, 32 bins a lane)
  if (warp == 0) {
    constexpr int kPer = kHistBins / 32;
    unsigned long long part = 0ull;
    for (int j = 0; j < kPer; ++j) part += hist_at(lane * kPer + j);
    unsigned long long inc = part;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    unsigned long long run = inc - part;
    int found = kHistBins;
    unsigned long long above = 0ull;
    for (int j = 0; j < kPer; ++j) {
      const unsigned long long h = hist_at(lane * kPer + j);
      if (found == kHistBins && h && (float)(run + h) / kFix >= target) {
        found = lane * kPer + j;
        above = run;
      }
      run += h;
    }
    int best = found;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (best == kHistBins) {   // rounding left the target just out of reach: the lowest populated bin
      int last = -1;
      for (int j = 0; j < kPer; ++j)
        if (hist_at(lane * kPer + j)) last = lane * kPer + j;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
      best = last;
      if (last >= lane * kPer && last < (lane + 1) * kPer) {
        unsigned long long a2 = inc - part;
        for (int j = lane * kPer; j < last; ++j) a2 += hist_at(j);
        found = last;
        above = a2;
      }
    }
    if (found == best) {
      s_bin = best;
      s_above = above;
    }
  }
  __syncthreads();
  const int tbin = s_bin;
  const float above = (float)s_above / kFix;
  // blocks above the bin are selected; those inside it become sort keys
#pragma unroll
  for (int k = 0; k < kMine; ++k) {
    const int i = tid + k * kSelThreads;
    if (i >= nb) continue;
    const float m = m_r[k];
    const int b = bin_of(m);
    if (b < tbin) {
      const int pos = atomicAdd(&s_n_above, 1);
      if (out_ids && pos < blk_stride) out_ids[pos] = i;
    } else if (b == tbin) {
      keys[atomicAdd(&s_n_in, 1)] = ((unsigned long long)(~okey(m)) << 32) | (unsigned long long)(uint32_t)i;
    }
  }
  __syncthreads();
  const int n_above = s_n_above, n_in = s_n_in;
  int np = 1;
  while (np < n_in) np <<= 1;
  for (int i = n_in + tid; i < np; i += kSelThreads) keys[i] = ~0ull;
  __syncthreads();
  // bitonic sort of the bin's blocks, ascending (usually a handful; all of the row's blocks when every maximum is equal)
  for (int size = 2; size <= np; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < (np >> 1); i += kSelThreads) {
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
  auto weight = [&](int i) -> float {   // mass of the i-th block of the bin's order, relative to exp(M)
    const unsigned long long k = keys[i];
    return mass_of(okey_to_float(~(uint32_t)(k >> 32)), lw[(uint32_t)k]);
  };
  for (int r0 = 0; r0 < n_in; r0 += kSelThreads) {
    if (s_pick != 0x7fffffff) break;   // uniform: written before the barrier that ends each round
    const int i = r0 + tid;
    const float e = i < n_in ? weight(i) : 0.f;
    float inc = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float a = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += a;
    }
    if (lane == 31) w_sum[warp] = inc;
    __syncthreads();
    float wbase = 0.f, tot = 0.f;
    for (int w = 0; w < kSelWarps; ++w) {
      if (w < warp) wbase += w_sum[w];
      tot += w_sum[w];
    }
    const float cum = above + s_run + wbase + inc;
    if (i < n_in && cum >= target) atomicMin(&s_pick, i);
    __syncthreads();
    if (i == s_pick) s_pick_mass = cum;
    if (tid == 0) s_run += tot;
    __syncthreads();
  }
  int pick = s_pick;
  float mass = s_pick_mass;
  if (pick == 0x7fffffff) {   // rounding left the target just out of reach: the whole bin
    pick = n_in - 1;
    mass = above + s_run;
  }
  const int c_in = pick + 1, c = n_above + c_in;
  if (out_ids) {
    for (int i = tid; i < c_in; i += kSelThreads)
      if (n_above + i < blk_stride) out_ids[n_above + i] = (int)(uint32_t)keys[i];
  }
  if (tid == 0) {
    const unsigned long long last = keys[c_in - 1];
    sel_count[rh] = c;
    if (sel_mass) sel_mass[rh] = Z > 0.f ? fminf(mass / Z, 1.0f) : 1.0f;
    if (sel_thresh) sel_thresh[rh] = c == nb ? -INFINITY : okey_to_float(~(uint32_t)(last >> 32));
    if (sel_tie_last) sel_tie_last[rh] = c == nb ? nb - 1 : (int)(uint32_t)last;
    if (out_ids && c > blk_stride) set_status(status, RTP_ERR_CAPACITY);
  }
}

// ---- union of the page lists of a KV head's query heads -------------------------------------------------------------
// One CTA per (row, KV head).  Every head's list is turned into a bit per page in shared memory; the union is written
// in increasing page order, each entry = page | (flags << 24), flag bit g = query head g of the group selected the page.
constexpr int kUniThreads = 1024;
constexpr int kUniLoads = 8;   // list entries a thread has in flight

__global__ void __launch_bounds__(kUniThreads) blk_union_kernel(const CacheView cv, const Dims d, const HeadMaps hm,
                                                                const Rows rows, const int32_t* __restrict__ blk_idx,
                                                                const int64_t blk_stride,
                                                                const int32_t* __restrict__ blk_cnt,
                                                                int32_t* __restrict__ uni_idx, const int64_t uni_stride,
                                                                int32_t* __restrict__ uni_cnt, const int nbw_max,
                                                                int32_t* status) {
  chain_wait();
  extern __shared__ uint32_t uni_bits[];   // [group][nbw_max]
  __shared__ int w_cnt[kUniThreads / 32];
  __shared__ int s_base;
  const int n_units = hm.n_kv_list;
  const int64_t r = blockIdx.x / n_units;
  const int u = blockIdx.x % n_units;
  const int kvh = hm.kv_list[u];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seq = rows.row_seq(r);
  int n_keys = rows.row_pos(r) + 1;
  {
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;
    n_keys = max(0, min(n_keys, sl));
  }
  const int nb = (n_keys + kPage - 1) >> kPageShift;
  const int nbw = (nb + 31) >> 5;
  __shared__ int s_cnt[8];                 // list length of head g of the group (0: not a retrieval head)
  __shared__ const int32_t* s_lst[8];
  for (int i = tid; i < d.group * nbw_max; i += kUniThreads) uni_bits[i] = 0u;
  if (tid == 0) s_base = 0;
  if (tid < 8) s_cnt[tid] = 0;
  __syncthreads();
  if (tid < d.n_ret) {
    const int qh = hm.ret_q_head[tid];
    if (qh / d.group == kvh) {
      const int64_t rh = r * d.n_ret + tid;
      s_cnt[qh % d.group] = max(0, (int)min((int64_t)__ldg(blk_cnt + rh), blk_stride));
      s_lst[qh % d.group] = blk_idx + rh * blk_stride;
    }
  }
  __syncthreads();
  int max_cnt = 0;
  for (int g = 0; g < d.group; ++g) max_cnt = max(max_cnt, s_cnt[g]);
  for (int j0 = tid; j0 < max_cnt; j0 += kUniThreads * kUniLoads) {
    for (int g = 0; g < d.group; ++g) {   // (the loads of a head are in flight together; heads follow each other closely)
      const int cnt = s_cnt[g];
      if (j0 - tid >= cnt) continue;      // uniform
      const int32_t* lst = s_lst[g];
      int page[kUniLoads];
#pragma unroll
      for (int k = 0; k < kUniLoads; ++k) {
        const int j = j0 + k * kUniThreads;
        page[k] = j < cnt ? __ldg(lst + j) : -1;
      }
#pragma unroll
      for (int k = 0; k < kUniLoads; ++k) {
        if (j0 + k * kUniThreads >= cnt) continue;
        if ((unsigned)page[k] >= (unsigned)nb) {
          set_status(status, RTP_ERR_INVALID);   // a page outside the row's causal pages is left out
          continue;
        }
        atomicOr(&uni_bits[g * nbw_max + (page[k] >> 5)], 1u << (page[k] & 31));
      }
    }
  }
  __syncthreads();
  int32_t* out = uni_idx + (int64_t)blockIdx.x * uni_stride;
  for (int w0 = 0; w0 < nbw; w0 += kUniThreads) {
    const int w = w0 + tid;
    uint32_t any = 0u;
    if (w < nbw)
      for (int g = 0; g < d.group; ++g) any |= uni_bits[g * nbw_max + w];
    const int mine = __popc(any);
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    if (lane == 31) w_cnt[warp] = inc;
    __syncthreads();
    int wbase = 0, tot = 0;
    for (int k = 0; k < kUniThreads / 32; ++k) {
      if (k < warp) wbase += w_cnt[k];
      tot += w_cnt[k];
    }
    int pos = s_base + wbase + inc - mine;
    while (any) {
      const int b = __ffs(any) - 1;
      any &= any - 1u;
      uint32_t flags = 0u;
      for (int g = 0; g < d.group; ++g) flags |= ((uni_bits[g * nbw_max + w] >> b) & 1u) << g;
      if (pos < uni_stride) out[pos] = (int32_t)((uint32_t)(w * 32 + b) | (flags << 24));
      ++pos;
    }
    __syncthreads();
    if (tid == 0) s_base += tot;
    __syncthreads();
  }
  if (tid == 0) uni_cnt[blockIdx.x] = min((int64_t)s_base, uni_stride);
}

int64_t blocks_padded(int64_t max_len) { return (((max_len + kPage - 1) / kPage) + 3) / 4 * 4; }

int stats_splits(const Dims& d, int64_t R, int64_t max_len, int sm_count) {
  const int64_t pages = (max_len + kPage - 1) / kPage;
  int64_t want = (4LL * sm_count + R * d.n_ih - 1) / (R * d.n_ih);
  const int64_t cap = (pages + 31) / 32;   // at least 32 pages per CTA
  int64_t s = want < cap ? want : cap;
  if (s < 1) s = 1;
  if (s > 4096) s = 4096;
  return (int)s;
}

}  // namespace

size_t select_rows_blocks_workspace_bytes(const Dims& d, int64_t R, int64_t max_len) {
  if (R <= 0 || d.n_ret <= 0) return 0;
  return (size_t)R * d.n_ret * blocks_padded(max_len) * sizeof(float2);
}

size_t block_union_bytes(const Dims& d, int64_t R, int64_t max_len) {
  if (R <= 0) return 0;
  return (size_t)R * d.n_kv * (blocks_padded(max_len) + 16) * sizeof(int32_t);
}

cudaError_t launch_block_union(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const int32_t* blk_idx, int64_t blk_stride, const int32_t* blk_cnt, int64_t max_len,
                               void* ws, int32_t** uni_idx, int64_t* uni_stride, int32_t** uni_cnt, int32_t* status,
                               cudaStream_t st) {
  const int64_t units = rows.R * hm.n_kv_list;
  const int64_t stride = blocks_padded(max_len);
  int32_t* idx = reinterpret_cast<int32_t*>(ws);
  int32_t* cnt = idx + units * stride;
  *uni_idx = idx;
  *uni_stride = stride;
  *uni_cnt = cnt;
  if (units == 0) return cudaSuccess;
  const int nbw_max = (int)((stride + 31) / 32);
  (void)launch_chained(blk_union_kernel, dim3((unsigned)units), dim3(kUniThreads), (size_t)d.group * nbw_max * 4, st, cv, d, hm,
                       rows, blk_idx, blk_stride, blk_cnt, idx, stride, cnt, nbw_max, status);
  return cudaGetLastError();
}

cudaError_t launch_select_rows_blocks(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                      const __nv_bfloat16* qt, int64_t max_len, int32_t* blk_idx, int64_t blk_stride,
                                      int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                      int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  const int64_t nb_pad = blocks_padded(max_len);
  const int64_t nb_max = (max_len + kPage - 1) / kPage;
  if (nb_max > kMaxBlocksRow) return cudaErrorNotSupported;
  float2* stats = reinterpret_cast<float2*>(ws);
  int max_nh = 0;
  for (int i = 0; i < d.n_ih; ++i) max_nh = hm.ih_nheads[i] > max_nh ? hm.ih_nheads[i] : max_nh;
  const int n_splits = stats_splits(d, rows.R, max_len, sm_count);
  const dim3 grid((unsigned)(rows.R * d.n_ih), n_splits);
#define RTP_STATS(NH4_, F8_) \
  (void)launch_chained(blk_stats_kernel<NH4_, F8_>, dim3(grid), dim3(kThreads), 0, st, cv, d, hm, rows, qt, stats, nb_pad, n_splits, status)
  if (max_nh <= 4) {
    if (cv.ikey_fp8) RTP_STATS(true, true); else RTP_STATS(true, false);
  } else {
    if (cv.ikey_fp8) RTP_STATS(false, true); else RTP_STATS(false, false);
  }
#undef RTP_STATS
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  int np2 = 1;
  while (np2 < nb_max) np2 <<= 1;
  const int smem = np2 * 8 + (int)nb_pad * 4;
  static PerDeviceOnce once;
  e = set_dyn_smem_once(blk_select_kernel, kMaxBlocksRow * 8 + kMaxBlocksRow * 4, once);
  if (e != cudaSuccess) return e;
  (void)launch_chained(blk_select_kernel, dim3((unsigned)(rows.R * d.n_ret)), dim3(kSelThreads), (size_t)smem, st, cv, d, rows,
                       stats, nb_pad, np2, blk_idx, blk_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status);
  return cudaGetLastError();
}

}  // namespace rtp
