// S2-S4 for explicit rows (the decode path): fused indexer scan + top-p selection (Eq. 5).
//
// The context of one (row, index head) is split over many CTAs.  Selection is a radix descent on
// the ordered 32-bit key of the fp32 score, with softmax mass as the weight:
//   hist pass    every CTA scores its keys (MMA, see score16) and adds exp(s - ref) and a count to a
//                2048-bin histogram of the next key bits (shared memory, then global atomics);
//   resolve      one CTA per (row, head) walks the bins from the top and finds the bucket in which the
//                cumulative mass reaches p * Z; as soon as that bucket holds <= kCandCap keys the row
//                stops refining;
//   compaction   every key above the bucket is emitted, keys inside it become candidates;
//   finalize     one CTA per (row, head) sorts the candidates by (score desc, position asc) and takes
//                the shortest prefix that reaches the target mass.
// The first histogram needs no row maximum: bin b accumulates exp(s - ub(b)) with ub(b) the largest
// value of the bin, and the resolve step rescales by exp(ub(b) - M) once M is known.
#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kHeadsPerCta = 4;
constexpr int kStage = 128;      // staged ids per (warp, head) before a flush
constexpr int kCandStage = 48;   // staged boundary candidates per (warp, head)

struct Bin {
  float mass;
  uint32_t cnt;
};

struct RowCtx {
  int64_t r;
  int ih, split, seq, n_keys, p_lo, p_hi, nh;
};

__device__ __forceinline__ RowCtx make_row_ctx(const CacheView& cv, const Dims& d, const HeadMaps& hm,
                                               const Rows& rows, int n_splits, int32_t* status) {
  RowCtx x;
  x.r = blockIdx.x / d.n_ih;
  x.ih = blockIdx.x % d.n_ih;
  x.split = blockIdx.y;
  x.nh = hm.ih_nheads[x.ih];
  x.seq = rows.row_seq(x.r);
  int n_keys = rows.row_pos(x.r) + 1;
  const int sl = (x.seq >= 0 && x.seq < cv.batch) ? cv.seq_lens[x.seq] : 0;
  if (n_keys > sl) {
    if (threadIdx.x == 0) set_status(status, RTP_ERR_INVALID);
    n_keys = sl;
  }
  if (n_keys < 0) n_keys = 0;
  x.n_keys = n_keys;
  const int n_pages = (n_keys + kPage - 1) >> kPageShift;
  const int per = (n_pages + n_splits - 1) / n_splits;
  x.p_lo = x.split * per;
  x.p_hi = min(n_pages, x.p_lo + per);
  return x;
}

// Which retrieval head (index into ret_q_heads) this lane post-processes in head group z, or -1.
// MMA row g holds head slot g, row g + 8 holds slot g + 8; group z covers slots 4z .. 4z+3.
__device__ __forceinline__ int lane_head_slot(int lane, int z) {
  const int g = lane >> 2;
  if ((g >> 2) != (z & 1)) return -1;
  return (z >> 1) * 8 + g;
}

__global__ void sel_init_kernel(const CacheView cv, const Dims d, const Rows rows, SelState* state,
                                int64_t n_rowheads) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_rowheads) return;
  const int64_t r = i / d.n_ret;
  const int seq = rows.row_seq(r);
  int n_keys = rows.row_pos(r) + 1;
  const int sl = (seq >= 0 && seq < cv.batch) ? cv.seq_lens[seq] : 0;
  n_keys = max(0, min(n_keys, sl));
  SelState s = {};
  s.n_keys = n_keys;
  s.mode = (d.top_p >= 1.0f || n_keys <= 1) ? kSelectAll : kRefine;
  s.hi_key = 0xffffffffu;
  state[i] = s;
}

// ---- histogram pass -----------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) sel_hist_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows,
    const __nv_bfloat16* __restrict__ qt, SelState* __restrict__ state, Bin* __restrict__ hist,
    int n_splits, int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* h_mass = reinterpret_cast<float*>(smem_raw);                              // [4][2048]
  uint32_t* h_cnt = reinterpret_cast<uint32_t*>(smem_raw + kHeadsPerCta * kSelBins * 4);  // [4][2048]
  __shared__ int any_active;

  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, status);
  const int z = blockIdx.z;
  if (z * kHeadsPerCta >= x.nh || x.p_lo >= x.p_hi) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, c = lane & 3;

  const int slot = lane_head_slot(lane, z);
  const bool use_hi = (z >> 1) != 0;
  const int j = (lane >> 2) & 3;
  int head = (slot >= 0 && slot < x.nh) ? hm.ih_heads[x.ih][slot] : -1;
  SelState* st = head >= 0 ? state + (x.r * d.n_ret + head) : nullptr;
  int level = 0, have_M = 0;
  uint32_t lo_key = 0;
  float M = 0.f;
  if (st) {
    if (st->mode != kRefine) {
      head = -1;
    } else {
      level = st->level;
      have_M = st->pad;
      lo_key = st->lo_key;
      M = st->M;
    }
  }
  if (threadIdx.x == 0) any_active = 0;
  __syncthreads();
  if (head >= 0) any_active = 1;
  __syncthreads();
  if (!any_active) return;
  for (int i = threadIdx.x; i < kHeadsPerCta * kSelBins; i += kThreads) {
    h_mass[i] = 0.f;
    h_cnt[i] = 0u;
  }
  __syncthreads();

  const QFrag qf = load_qfrag(qt + x.r * d.n_ret * kIndexDim, hm.ih_heads[x.ih], x.nh, lane);
  uint32_t max_key = 0;
  for (int p = x.p_lo + warp; p < x.p_hi; p += kWarps) {
    const __nv_bfloat16* base = ikey_page_ptr(cv, x.seq, p, x.ih);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = ld_stream_v4(base + (i * 32 + lane) * 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s_lo[4], s_hi[4];
      score16(qf, v[i], lane, s_lo, s_hi);
      if (head < 0) continue;
      const int n0 = p * kPage + i * 16 + 4 * c;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (n0 + e >= x.n_keys) continue;
        const float s = finish_score(use_hi ? s_hi[e] : s_lo[e], d.score_scale);
        const uint32_t key = okey(s);
        int bin;
        float ref = M;
        if (level == 0) {
          bin = key >> 21;
          max_key = max(max_key, key);
          if (!have_M) ref = okey_to_float((key | 0x1fffffu));
        } else if (level == 11) {
          if ((key ^ lo_key) >> 21) continue;
          bin = (key >> 10) & 0x7ff;
        } else {
          if ((key ^ lo_key) >> 10) continue;
          bin = key & 0x3ff;
        }
        atomicAdd(&h_mass[j * kSelBins + bin], __expf(s - ref));
        atomicAdd(&h_cnt[j * kSelBins + bin], 1u);
      }
    }
  }
  max_key = max(max_key, __shfl_xor_sync(0xffffffffu, max_key, 1));
  max_key = max(max_key, __shfl_xor_sync(0xffffffffu, max_key, 2));
  if (level == 0 && head >= 0 && c == 0 && max_key) atomicMax(&st->max_key, max_key);
  __syncthreads();
  for (int i = threadIdx.x; i < kHeadsPerCta * kSelBins; i += kThreads) {
    const uint32_t n = h_cnt[i];
    if (n == 0) continue;
    const int jj = i / kSelBins, bin = i % kSelBins;
    const int slot2 = (z >> 1) * 8 + (z & 1) * 4 + jj;  // head slot of entry jj in group z
    if (slot2 >= x.nh) continue;
    const int hd = hm.ih_heads[x.ih][slot2];
    Bin* b = hist + (x.r * d.n_ret + hd) * kSelBins + bin;
    atomicAdd(&b->mass, h_mass[i]);
    atomicAdd(&b->cnt, n);
  }
}

// ---- resolve --------------------------------------------------------------------------------------
constexpr int kResThreads = 256;

__global__ void __launch_bounds__(kResThreads) sel_resolve_kernel(const Dims d, SelState* __restrict__ state,
                                                                  Bin* __restrict__ hist) {
  SelState* st = state + blockIdx.x;
  if (st->mode != kRefine) return;
  Bin* bins = hist + (int64_t)blockIdx.x * kSelBins;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int level = st->level;
  const int have_M = st->pad;
  const int nb = (level == 22) ? 1024 : kSelBins;
  const float M = (level == 0 && !have_M) ? okey_to_float(st->max_key) : st->M;
  __shared__ float w_mass[kResThreads / 32];
  __shared__ uint32_t w_cnt[kResThreads / 32];
  __shared__ int s_wide, s_found, s_last;
  if (tid == 0) {
    s_wide = 0;
    s_found = 0x7fffffff;
    s_last = -1;
  }
  __syncthreads();

  float mass[8];
  uint32_t cnt[8];
  float tm = 0.f;
  uint32_t tc = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int o = tid * 8 + k;  // order index: 0 = top bin
    mass[k] = 0.f;
    cnt[k] = 0;
    if (o < nb) {
      const int bin = nb - 1 - o;
      const Bin b = bins[bin];
      bins[bin] = Bin{0.f, 0u};
      cnt[k] = b.cnt;
      float m = b.mass;
      if (level == 0 && !have_M && b.cnt) {
        const uint32_t ubk = ((uint32_t)bin << 21) | 0x1fffffu;
        const uint32_t ex = (ubk & 0x80000000u) ? ((ubk >> 23) & 0xff) : ((~ubk >> 23) & 0xff);
        if (ex >= 127 + 8) s_wide = 1;
        m *= __expf(okey_to_float(ubk) - M);
      }
      mass[k] = m;
      tm += m;
      tc += b.cnt;
    }
  }
  __syncthreads();
  if (s_wide) {  // very large scores: the bin-relative masses may have underflowed; redo relative to M
    if (tid == 0) {
      st->M = M;
      st->pad = 1;
    }
    return;
  }
  // block exclusive scan of (tm, tc) in order of tid
  float im = tm;
  uint32_t ic = tc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float a = __shfl_up_sync(0xffffffffu, im, o);
    const uint32_t b = __shfl_up_sync(0xffffffffu, ic, o);
    if (lane >= o) {
      im += a;
      ic += b;
    }
  }
  if (lane == 31) {
    w_mass[warp] = im;
    w_cnt[warp] = ic;
  }
  __syncthreads();
  float base_m = 0.f, total_m = 0.f;
  uint32_t base_c = 0;
  for (int w = 0; w < kResThreads / 32; ++w) {
    if (w < warp) {
      base_m += w_mass[w];
      base_c += w_cnt[w];
    }
    total_m += w_mass[w];
  }
  float ex_m = base_m + im - tm;  // mass of bins before this thread's first bin
  uint32_t ex_c = base_c + ic - tc;

  float Z = st->Z, target = st->target;
  if (level == 0) {
    Z = total_m;
    target = d.top_p * Z * (1.0f + kMassMargin);
  }
  const float above0 = st->mass_above;
  // first bin (from the top) at which the cumulative mass reaches the target
  {
    float run = ex_m;
    int found = -1, last = -1;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (cnt[k]) {
        last = tid * 8 + k;
        if (found < 0 && above0 + run + mass[k] >= target) found = tid * 8 + k;
      }
      run += mass[k];
    }
    if (found >= 0) atomicMin(&s_found, found);
    if (last >= 0) atomicMax(&s_last, last);
  }
  __syncthreads();
  int pick = s_found;
  if (pick == 0x7fffffff) pick = s_last;  // rounding left the target just out of reach: take everything
  if (pick < 0) return;                   // empty histogram (cannot happen for a non-empty row)
  if (pick / 8 == tid) {
    float run = ex_m;
    uint32_t runc = ex_c;
    for (int k = 0; k < (pick & 7); ++k) {
      run += mass[k];
      runc += cnt[k];
    }
    const int k = pick & 7;
    const uint32_t bin = (uint32_t)(nb - 1 - pick);
    uint32_t lo, hi;
    int new_level;
    if (level == 0) {
      lo = bin << 21;
      hi = lo | 0x1fffffu;
      new_level = 11;
    } else if (level == 11) {
      lo = (st->lo_key & 0xffe00000u) | (bin << 10);
      hi = lo | 0x3ffu;
      new_level = 22;
    } else {
      lo = (st->lo_key & 0xfffffc00u) | bin;
      hi = lo;
      new_level = 32;
    }
    st->lo_key = lo;
    st->hi_key = hi;
    st->level = new_level;
    st->M = M;
    st->Z = Z;
    st->target = target;
    st->mass_above = above0 + run;
    st->cnt_above = st->cnt_above + (int)runc;
    st->bucket_cnt = (int)cnt[k];
    st->bucket_mass = mass[k];
    st->pad = 1;
    if ((int)cnt[k] <= kCandCap)
      st->mode = kCollect;
    else if (new_level == 32)
      st->mode = kTieScan;
  }
}

// ---- compaction -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) sel_compact_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows,
    const __nv_bfloat16* __restrict__ qt, SelState* __restrict__ state, uint2* __restrict__ cand,
    int32_t* __restrict__ sel_idx, int64_t sel_stride, int n_splits, int32_t* status) {
  __shared__ int stage[kWarps][kHeadsPerCta][kStage];
  __shared__ uint2 cstage[kWarps][kHeadsPerCta][kCandStage];
  __shared__ int stage_cnt[kWarps][kHeadsPerCta];
  __shared__ int cstage_cnt[kWarps][kHeadsPerCta];

  const RowCtx x = make_row_ctx(cv, d, hm, rows, n_splits, nullptr);
  const int z = blockIdx.z;
  if (z * kHeadsPerCta >= x.nh || x.p_lo >= x.p_hi) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, c = lane & 3;
  const int slot = lane_head_slot(lane, z);
  const bool use_hi = (z >> 1) != 0;
  const int j = (lane >> 2) & 3;
  const int head = (slot >= 0 && slot < x.nh) ? hm.ih_heads[x.ih][slot] : -1;
  SelState* st = head >= 0 ? state + (x.r * d.n_ret + head) : nullptr;
  int mode = -1;
  uint32_t lo_key = 0, hi_key = 0;
  if (st) {
    mode = st->mode;
    lo_key = st->lo_key;
    hi_key = st->hi_key;
  }
  if (lane < kHeadsPerCta) {
    stage_cnt[warp][lane] = 0;
    cstage_cnt[warp][lane] = 0;
  }
  __syncwarp();
  const bool emit_ids = sel_idx != nullptr;
  const QFrag qf = load_qfrag(qt + x.r * d.n_ret * kIndexDim, hm.ih_heads[x.ih], x.nh, lane);

  auto row_head = [&](int jj) -> int64_t {
    const int slot2 = (z >> 1) * 8 + (z & 1) * 4 + jj;
    return x.r * d.n_ret + hm.ih_heads[x.ih][slot2];
  };
  auto flush_ids = [&](int jj) {  // warp-uniform
    const int n = stage_cnt[warp][jj];
    if (n == 0) return;
    const int64_t rh = row_head(jj);
    int gbase = 0;
    if (lane == 0) gbase = atomicAdd(&state[rh].emit_cnt, n);
    gbase = __shfl_sync(0xffffffffu, gbase, 0);
    for (int i = lane; i < n; i += 32)
      if (gbase + i < sel_stride) sel_idx[rh * sel_stride + gbase + i] = stage[warp][jj][i];
    if (gbase + n > sel_stride && lane == 0) set_status(status, RTP_ERR_CAPACITY);
    __syncwarp();
    if (lane == 0) stage_cnt[warp][jj] = 0;
    __syncwarp();
  };
  auto flush_cands = [&](int jj) {  // warp-uniform
    const int n = cstage_cnt[warp][jj];
    if (n == 0) return;
    const int64_t rh = row_head(jj);
    int gbase = 0;
    if (lane == 0) gbase = atomicAdd(&state[rh].cand_cnt, n);
    gbase = __shfl_sync(0xffffffffu, gbase, 0);
    for (int i = lane; i < n; i += 32)
      if (gbase + i < kCandCap) cand[rh * kCandCap + gbase + i] = cstage[warp][jj][i];
    __syncwarp();
    if (lane == 0) cstage_cnt[warp][jj] = 0;
    __syncwarp();
  };
  // Appends the entries flagged in `flags` (bit e = key n0 + e) of every head to a per-warp stage.
  auto group_offsets = [&](int k, int& incl) {
    incl = k;
    int t = __shfl_up_sync(0xffffffffu, incl, 1, 4);
    if (c >= 1) incl += t;
    t = __shfl_up_sync(0xffffffffu, incl, 2, 4);
    if (c >= 2) incl += t;
  };

  for (int p = x.p_lo + warp; p < x.p_hi; p += kWarps) {
    const __nv_bfloat16* base = ikey_page_ptr(cv, x.seq, p, x.ih);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = ld_stream_v4(base + (i * 32 + lane) * 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s_lo[4], s_hi[4];
      score16(qf, v[i], lane, s_lo, s_hi);
      const int n0 = p * kPage + i * 16 + 4 * c;
      int flags = 0, cflags = 0;
      uint32_t keys4[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) keys4[e] = okey(finish_score(use_hi ? s_hi[e] : s_lo[e], d.score_scale));
      if (mode == kSelectAll) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (n0 + e < x.n_keys) flags |= 1 << e;
      } else if (mode == kCollect || mode == kTieScan) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (n0 + e >= x.n_keys) continue;
          if (keys4[e] > hi_key)
            flags |= 1 << e;
          else if (keys4[e] >= lo_key && mode == kCollect)
            cflags |= 1 << e;
        }
      }
      // boundary candidates
      {
        const int k = __popc(cflags);
        int incl;
        group_offsets(k, incl);
        if (head >= 0 && k) {
          int w = cstage_cnt[warp][j] + incl - k;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (cflags & (1 << e)) cstage[warp][j][w++] = make_uint2(keys4[e], (uint32_t)(n0 + e));
        }
        __syncwarp();
        if (head >= 0 && c == 3 && incl) cstage_cnt[warp][j] += incl;
        __syncwarp();
#pragma unroll
        for (int jj = 0; jj < kHeadsPerCta; ++jj)
          if (cstage_cnt[warp][jj] > kCandStage - 16) flush_cands(jj);
      }
      if (!emit_ids) continue;
      {
        const int k = __popc(flags);
        int incl;
        group_offsets(k, incl);
        if (head >= 0 && k) {
          int w = stage_cnt[warp][j] + incl - k;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (flags & (1 << e)) stage[warp][j][w++] = n0 + e;
        }
        __syncwarp();
        if (head >= 0 && c == 3 && incl) stage_cnt[warp][j] += incl;
        __syncwarp();
#pragma unroll
        for (int jj = 0; jj < kHeadsPerCta; ++jj)
          if (stage_cnt[warp][jj] > kStage - 16) flush_ids(jj);
      }
    }
  }
#pragma unroll
  for (int jj = 0; jj < kHeadsPerCta; ++jj) {
    flush_cands(jj);
    if (emit_ids) flush_ids(jj);
  }
}

// ---- finalize ---------------------------------------------------------------------------------------
constexpr int kFinThreads = 256;
constexpr int kFinWarps = kFinThreads / 32;
constexpr int kNoPick = 0x7fffffff;

__global__ void __launch_bounds__(kFinThreads) sel_finalize_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows,
    const __nv_bfloat16* __restrict__ qt, SelState* __restrict__ state, const uint2* __restrict__ cand,
    int32_t* __restrict__ sel_idx, int64_t sel_stride, int32_t* __restrict__ sel_count,
    float* __restrict__ sel_mass, float* __restrict__ sel_thresh, int32_t* __restrict__ sel_tie_last,
    int32_t* status) {
  __shared__ unsigned long long keys[kCandCap];  // 32 KB
  __shared__ float w_sum[kFinWarps];
  __shared__ int w_cnt[kFinWarps];
  __shared__ int s_pick, s_emitted, s_last;
  __shared__ float s_run, s_pick_mass;
  const int64_t rh = blockIdx.x;
  SelState* st = state + rh;
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
  const float M = st->M, Z = st->Z, target = st->target, above = st->mass_above;
  const int base = st->cnt_above;
  const int emit_base = ids ? st->emit_cnt : base;

  if (mode == kCollect) {
    const int n = min(st->cand_cnt, kCandCap);
    int np = 1;
    while (np < n) np <<= 1;
    for (int i = tid; i < np; i += kFinThreads) {
      unsigned long long k = ~0ull;
      if (i < n) {
        const uint2 cnd = cand[rh * kCandCap + i];
        k = ((unsigned long long)(~cnd.x) << 32) | (unsigned long long)cnd.y;
      }
      keys[i] = k;
    }
    if (tid == 0) {
      s_pick = kNoPick;
      s_run = 0.f;
      s_pick_mass = 0.f;
    }
    __syncthreads();
    // bitonic sort, ascending: larger score first, then smaller position
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
      if (i < n) e = __expf(okey_to_float(~(uint32_t)(keys[i] >> 32)) - M);
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
    if (tid == 0) {
      sel_count[rh] = base + c;
      if (sel_mass) sel_mass[rh] = mass / Z;
      if (sel_thresh) sel_thresh[rh] = okey_to_float(~(uint32_t)(keys[pick] >> 32));
      if (sel_tie_last) sel_tie_last[rh] = (int)(uint32_t)keys[pick];
      if (ids && base + c > sel_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }

  if (mode == kTieScan) {
    // More than kCandCap keys share the threshold score exactly: take the first c of them in
    // position order, c = the number of equal masses still needed.
    const uint32_t t_key = st->lo_key;
    const float e_t = __expf(okey_to_float(t_key) - M);
    int c = (int)ceilf((target - above) / e_t);
    c = max(1, min(c, st->bucket_cnt));
    const int64_t r = rh / d.n_ret;
    const int head = (int)(rh % d.n_ret);
    const int ih = hm.q2ih[head];
    const int slot = hm.slot_in_ih[head];
    const int seq = rows.row_seq(r);
    const QFrag qf = load_qfrag(qt + r * d.n_ret * kIndexDim, hm.ih_heads[ih], hm.ih_nheads[ih], lane);
    unsigned char* flags = reinterpret_cast<unsigned char*>(keys);  // [kFinWarps * 64]
    if (tid == 0) {
      s_emitted = 0;
      s_last = -1;
    }
    __syncthreads();
    const int n_pages = (n_keys + kPage - 1) >> kPageShift;
    for (int p0 = 0; p0 < n_pages; p0 += kFinWarps) {
      if (s_emitted >= c) break;  // uniform (see barrier at the end of the round)
      const int p = p0 + warp;
      if (p < n_pages) {
        const __nv_bfloat16* pb = ikey_page_ptr(cv, seq, p, ih);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 v = ld_stream_v4(pb + (i * 32 + lane) * 8);
          float s_lo[4], s_hi[4];
          score16(qf, v, lane, s_lo, s_hi);
          if ((lane >> 2) == (slot & 7)) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int n = p * kPage + i * 16 + 4 * (lane & 3) + e;
              const uint32_t key = okey(finish_score((slot >> 3) ? s_hi[e] : s_lo[e], d.score_scale));
              flags[warp * kPage + i * 16 + 4 * (lane & 3) + e] = (n < n_keys && key == t_key) ? 1 : 0;
            }
          }
        }
      } else {
        for (int i = lane; i < kPage; i += 32) flags[warp * kPage + i] = 0;
      }
      __syncthreads();
      // ordered emission: thread t owns keys 2t, 2t+1 of this round
      const int f0 = flags[2 * tid], f1 = flags[2 * tid + 1];
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
      const int n_first = p0 * kPage + 2 * tid;
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
    if (tid == 0) {
      sel_count[rh] = base + c;
      if (sel_mass) sel_mass[rh] = (above + (float)c * e_t) / Z;
      if (sel_thresh) sel_thresh[rh] = okey_to_float(t_key);
      if (sel_tie_last) sel_tie_last[rh] = s_last;
      if (ids && base + c > sel_stride) set_status(status, RTP_ERR_CAPACITY);
    }
    return;
  }
  // still refining after every level: cannot happen (three levels resolve all 32 key bits)
  if (tid == 0) {
    sel_count[rh] = 0;
    set_status(status, RTP_ERR_UNSUPPORTED);
  }
}

int select_splits(const Dims& d, int64_t R, int64_t max_len, int sm_count) {
  const int64_t pages = (max_len + kPage - 1) / kPage;
  int64_t want = (4LL * sm_count + R * d.n_ih - 1) / (R * d.n_ih);
  int64_t cap = (pages + 31) / 32;  // at least 32 pages (2048 keys) per CTA
  int64_t s = want < cap ? want : cap;
  if (s < 1) s = 1;
  if (s > 4096) s = 4096;
  return (int)s;
}

struct SelWorkspace {
  SelState* state;
  Bin* hist;
  uint2* cand;
  size_t bytes;
};

SelWorkspace carve(void* ws, int64_t n_rowheads) {
  SelWorkspace w;
  size_t off = 0;
  auto take = [&](size_t n) {
    size_t o = off;
    off += (n + 255) & ~(size_t)255;
    return o;
  };
  const size_t o_state = take(sizeof(SelState) * n_rowheads);
  const size_t o_hist = take(sizeof(Bin) * kSelBins * n_rowheads);
  const size_t o_cand = take(sizeof(uint2) * kCandCap * n_rowheads);
  char* b = reinterpret_cast<char*>(ws);
  w.state = reinterpret_cast<SelState*>(b + o_state);
  w.hist = reinterpret_cast<Bin*>(b + o_hist);
  w.cand = reinterpret_cast<uint2*>(b + o_cand);
  w.bytes = off;
  return w;
}

}  // namespace

size_t select_rows_workspace_bytes(const Dims& d, int64_t R) {
  if (R <= 0 || d.n_ret <= 0) return 0;
  return carve(nullptr, R * d.n_ret).bytes;
}

cudaError_t launch_select_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const __nv_bfloat16* qt, int64_t max_len, int32_t* sel_idx, int64_t sel_stride,
                               int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                               int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  const int64_t nrh = rows.R * d.n_ret;
  const SelWorkspace w = carve(ws, nrh);
  cudaError_t e = cudaMemsetAsync(w.hist, 0, sizeof(Bin) * kSelBins * nrh, st);
  if (e != cudaSuccess) return e;
  sel_init_kernel<<<(unsigned)((nrh + 127) / 128), 128, 0, st>>>(cv, d, rows, w.state, nrh);
  int max_nh = 0;
  for (int i = 0; i < d.n_ih; ++i) max_nh = hm.ih_nheads[i] > max_nh ? hm.ih_nheads[i] : max_nh;
  const int n_splits = select_splits(d, rows.R, max_len, sm_count);
  dim3 grid((unsigned)(rows.R * d.n_ih), n_splits, (max_nh + kHeadsPerCta - 1) / kHeadsPerCta);
  const size_t hist_smem = (size_t)kHeadsPerCta * kSelBins * 8;
  static bool attr_done = false;
  if (!attr_done) {
    e = cudaFuncSetAttribute(sel_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hist_smem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  for (int it = 0; it < 4; ++it) {
    sel_hist_kernel<<<grid, kThreads, hist_smem, st>>>(cv, d, hm, rows, qt, w.state, w.hist, n_splits, status);
    sel_resolve_kernel<<<(unsigned)nrh, kResThreads, 0, st>>>(d, w.state, w.hist);
  }
  sel_compact_kernel<<<grid, kThreads, 0, st>>>(cv, d, hm, rows, qt, w.state, w.cand, sel_idx, sel_stride,
                                                n_splits, status);
  sel_finalize_kernel<<<(unsigned)nrh, kFinThreads, 0, st>>>(cv, d, hm, rows, qt, w.state, w.cand, sel_idx,
                                                             sel_stride, sel_count, sel_mass, sel_thresh,
                                                             sel_tie_last, status);
  return cudaGetLastError();
}

}  // namespace rtp
