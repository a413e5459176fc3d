// S6 / S7 / S9 for a prefill chunk: tiled causal attention on tensor cores.
//
// One CTA owns 128 MMA rows = (128 / G) consecutive query positions x the G query heads of one KV
// head, so that every K/V tile fetched from the paged cache serves the whole GQA group.  Key tiles
// are pages (64 keys x 128 dims, 16 KB contiguous per KV head), double-buffered with cp.async and
// swizzled in shared memory; QK^T and PV run as bf16 m16n8k16 MMAs with fp32 accumulation and an
// online softmax per row.
//   dense   every tile up to the diagonal                                   (comparator, S9)
//   local   the sink tile(s) plus the tiles that intersect (m - W, m]       (Section 3.2, S7)
//   sparse  every tile up to the diagonal; membership of (row, key) in S_h(m) is re-evaluated from
//           the 16-dim indexer score and the row's (threshold, tie position) pair, and a warp skips
//           the two big MMAs of a tile in which none of its rows selects a key     (Eq. 5, S6)
#include <cstdlib>

#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kRows = 128;            // MMA rows per CTA
constexpr int kWarpsP = 8;
constexpr int kThreadsP = kWarpsP * 32;
constexpr int kBN = kPage;            // keys per tile
constexpr int kStages = 2;
constexpr int kTileBytes = kBN * kHeadDim * 2;          // 16 KB
constexpr int kIkTileBytes = kBN * kIndexDim * 2;       // 2 KB
constexpr int kQBytes = kRows * kHeadDim * 2;           // 32 KB
constexpr int kSmemBytes = kQBytes + kStages * (2 * kTileBytes + kIkTileBytes);
constexpr float kLog2eP = 1.4426950408889634f;
constexpr float kLn2P = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
// Byte offset of 16-byte chunk `ch` of row `row` in a [rows][128] bf16 tile (256-byte rows), swizzled.
__device__ __forceinline__ int swz(int row, int ch) { return row * 256 + ((ch ^ (row & 7)) << 4); }

template <int G, int MODE>
__global__ void __launch_bounds__(kThreadsP, 2) attn_prefill_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const __nv_bfloat16* __restrict__ q,
    const __nv_bfloat16* __restrict__ qt, const int seq_id, const int q_start, const int C,
    const float* __restrict__ sel_thresh, const int32_t* __restrict__ sel_tie_last,
    __nv_bfloat16* __restrict__ out, float* __restrict__ lse, const int n_row_tiles) {
  constexpr int BMP = kRows / G;   // query positions per CTA
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* q_s = smem;
  unsigned char* kv_s = smem + kQBytes;   // per stage: K tile, V tile, index-key tile
  constexpr int kStageBytes = 2 * kTileBytes + kIkTileBytes;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, c = lane & 3;
  const int tile = n_row_tiles - 1 - blockIdx.x;   // heaviest (latest) row tiles first
  const int kvh = (MODE == kPrefillSparse) ? hm.ih_kv[blockIdx.y] : hm.kv_list[blockIdx.y];
  const int r0 = tile * BMP;                        // first chunk row of the CTA
  const int m0 = q_start + r0;                      // its position
  const int rows_here = min(BMP, C - r0);
  const int m_last = m0 + rows_here - 1;

  // rows of this warp: 16 consecutive MMA rows = one head, 16 consecutive positions
  const int wrow = warp * 16;
  const int hslot = wrow / BMP;                     // head of the group
  const int pofs = wrow % BMP;                      // position offset inside the CTA tile
  const int qh = kvh * d.group + hslot;

  // ---- Q tile -> shared (rows = [head][position]) ----
  for (int i = tid; i < kRows * 16; i += kThreadsP) {
    const int row = i >> 4, ch = i & 15;
    const int hs = row / BMP, po = row % BMP;
    const bool ok = po < rows_here;
    const __nv_bfloat16* src = q + ((int64_t)(r0 + (ok ? po : 0)) * d.n_q + kvh * d.group + hs) * kHeadDim + ch * 8;
    cp_async16(smem_u32(q_s + swz(row, ch)), src, ok);
  }
  cp_async_commit();

  // ---- key tiles visited by this CTA ----
  const int kt_last = m_last >> kPageShift;
  int n_sink_tiles = 0, kt_first = 0;
  if (MODE == kPrefillLocal) {
    kt_first = max(0, m0 - d.window + 1) >> kPageShift;
    n_sink_tiles = min((d.n_sink + kBN - 1) >> kPageShift, kt_first);
  }
  const int n_tiles = n_sink_tiles + (kt_last - kt_first + 1);
  auto tile_at = [&](int i) { return i < n_sink_tiles ? i : kt_first + (i - n_sink_tiles); };

  const int64_t bt_base = (int64_t)seq_id * cv.max_pages;
  const int ih = (MODE == kPrefillSparse) ? blockIdx.y : 0;
  auto load_tile = [&](int i, int stage) {
    const int kt = tile_at(i);
    const int phys = __ldg(cv.block_table + bt_base + kt);
    unsigned char* st = kv_s + stage * kStageBytes;
    const __nv_bfloat16* ksrc = cv.k + ((int64_t)phys * cv.n_kv + kvh) * (kBN * kHeadDim);
    const __nv_bfloat16* vsrc = cv.v + ((int64_t)phys * cv.n_kv + kvh) * (kBN * kHeadDim);
    const int n_ok = m_last - kt * kBN + 1;   // keys of this tile that any row may attend
#pragma unroll
    for (int x = 0; x < (kBN * 16) / kThreadsP; ++x) {
      const int i2 = tid + x * kThreadsP;
      const int row = i2 >> 4, ch = i2 & 15;
      const bool ok = row < n_ok;
      cp_async16(smem_u32(st + swz(row, ch)), ksrc + row * kHeadDim + ch * 8, ok);
      cp_async16(smem_u32(st + kTileBytes + swz(row, ch)), vsrc + row * kHeadDim + ch * 8, ok);
    }
    if (MODE == kPrefillSparse) {
      if (tid < kIkTileBytes / 16) {
        const __nv_bfloat16* isrc = cv.ikey + ((int64_t)phys * cv.n_ih + ih) * (kBN * kIndexDim);
        cp_async16(smem_u32(st + 2 * kTileBytes + tid * 16), isrc + tid * 8, true);
      }
    }
  };

  load_tile(0, 0);
  cp_async_commit();

  // ---- wait for Q ----
  cp_async_wait<1>();
  __syncthreads();
  // Q fragments are re-read from shared memory at every k-step (keeping them in registers spills)
  const uint32_t q_row_u32 = smem_u32(q_s) + (wrow + (lane & 7) + ((lane >> 3) & 1) * 8) * 256;
  const int q_row7 = (wrow + (lane & 7) + ((lane >> 3) & 1) * 8) & 7;

  // positions of the two rows this lane owns (g and g + 8 of the warp's 16)
  const int pos_a = m0 + pofs + g, pos_b = pos_a + 8;
  const bool row_a_ok = pofs + g < rows_here, row_b_ok = pofs + g + 8 < rows_here;
  const int warp_m_lo = m0 + pofs, warp_m_hi = min(m0 + pofs + 15, m_last);

  // sparse mode: projected query fragment and the rows' membership rule
  QFrag iq = {0u, 0u, 0u, 0u};
  // Membership is tested on the unscaled MMA output: raw > up_x means "score above the threshold", raw >= lo_x
  // means "score at or above it" (the two differ only for keys tied with the threshold score).
  const float kInfP = __int_as_float(0x7f800000);
  float lo_a = kInfP, up_a = kInfP, lo_b = kInfP, up_b = kInfP;
  int tie_a = -1, tie_b = -1;
  if (MODE == kPrefillSparse) {
    const int rh = hm.ih_heads[ih][hslot];   // retrieval-head index of this warp's head
    const int off = qfrag_dim_offset(lane);
    if (row_a_ok) {
      const int64_t rr = (int64_t)(r0 + pofs + g) * d.n_ret + rh;
      const uint2 v = *reinterpret_cast<const uint2*>(qt + rr * kIndexDim + off);
      iq.a0 = v.x;
      iq.a2 = v.y;
      const uint32_t tk = okey(sel_thresh[rr]);
      float dummy;
      raw_preimage(d.score_scale, tk, tk, lo_a, dummy);
      raw_preimage(d.score_scale, 0u, tk, dummy, up_a);
      tie_a = sel_tie_last[rr];
    }
    if (row_b_ok) {
      const int64_t rr = (int64_t)(r0 + pofs + g + 8) * d.n_ret + rh;
      const uint2 v = *reinterpret_cast<const uint2*>(qt + rr * kIndexDim + off);
      iq.a1 = v.x;
      iq.a3 = v.y;
      const uint32_t tk = okey(sel_thresh[rr]);
      float dummy;
      raw_preimage(d.score_scale, tk, tk, lo_b, dummy);
      raw_preimage(d.score_scale, 0u, tk, dummy, up_b);
      tie_b = sel_tie_last[rr];
    }
  }

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float mx_a = -INFINITY, mx_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  const float sc2 = d.sm_scale * kLog2eP;

  for (int it = 0; it < n_tiles; ++it) {
    const int stage = it & 1;
    if (it + 1 < n_tiles) load_tile(it + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();

    const int kt = tile_at(it);
    const int n_base = kt * kBN;
    unsigned char* st = kv_s + stage * kStageBytes;
    const uint32_t k_u32 = smem_u32(st), v_u32 = smem_u32(st + kTileBytes);

    // does this warp take part in the tile at all?
    bool active = n_base <= warp_m_hi;
    if (MODE == kPrefillLocal) active = active && (n_base + kBN - 1 > warp_m_lo - d.window || n_base < d.n_sink);
    // membership bits of the 32 S elements this lane owns (sparse mode)
    uint32_t member = 0xffffffffu;
    if (MODE == kPrefillSparse && active) {
      member = 0;
      const bool easy = (n_base + kBN - 1 <= warp_m_lo) &&
                        __all_sync(0xffffffffu, (!row_a_ok || tie_a >= n_base + kBN - 1) && (!row_b_ok || tie_b >= n_base + kBN - 1));
      const unsigned char* ik = st + 2 * kTileBytes;
      const int boff = 2 * qfrag_dim_offset(lane);
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const uint2 b = *reinterpret_cast<const uint2*>(ik + (nt * 8 + g) * (kIndexDim * 2) + boff);
        const float zero[4] = {0.f, 0.f, 0.f, 0.f};
        float s4[4];
        mma_bf16_16816(s4, iq.a0, iq.a1, iq.a2, iq.a3, b.x, b.y, zero);
        if (easy) {
          // every key of the tile is causal for every row of the warp and lies at or before the rows' tie positions
          member |= (s4[0] >= lo_a ? 1u : 0u) << (nt * 4) | (s4[1] >= lo_a ? 1u : 0u) << (nt * 4 + 1) |
                    (s4[2] >= lo_b ? 1u : 0u) << (nt * 4 + 2) | (s4[3] >= lo_b ? 1u : 0u) << (nt * 4 + 3);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int n = n_base + nt * 8 + 2 * c + (e & 1);
            const bool lo_row = e < 2;
            const float raw = s4[e];
            const bool in = (n <= (lo_row ? pos_a : pos_b)) &&
                            (raw > (lo_row ? up_a : up_b) || (raw >= (lo_row ? lo_a : lo_b) && n <= (lo_row ? tie_a : tie_b)));
            member |= (in ? 1u : 0u) << (nt * 4 + e);
          }
        }
      }
      active = __any_sync(0xffffffffu, member != 0);
    }

    if (active) {
      // ---- S = Q K^T ----
      float s[8][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t qa[4];
        ldmatrix_x4(qa, q_row_u32 + (((ks * 2 + (lane >> 4)) ^ q_row7) << 4));
#pragma unroll
        for (int np = 0; np < 4; ++np) {   // pairs of n8 tiles
          uint32_t b[4];
          const int row = np * 16 + (lane & 7) + (lane >> 4) * 8;
          const int ch = ks * 2 + ((lane >> 3) & 1);
          ldmatrix_x4(b, k_u32 + swz(row, ch));
          mma_bf16_16816(s[2 * np], qa[0], qa[1], qa[2], qa[3], b[0], b[1], s[2 * np]);
          mma_bf16_16816(s[2 * np + 1], qa[0], qa[1], qa[2], qa[3], b[2], b[3], s[2 * np + 1]);
        }
      }
      // ---- mask ----
      bool need_mask = n_base + kBN - 1 > warp_m_lo;   // tile reaches past the first row's diagonal
      if (MODE == kPrefillLocal) need_mask = need_mask || (n_base <= warp_m_hi - d.window);
      if (MODE == kPrefillSparse) need_mask = true;
      if (need_mask) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int n = n_base + nt * 8 + 2 * c + (e & 1);
            const int pos = e < 2 ? pos_a : pos_b;
            bool ok = n <= pos;
            if (MODE == kPrefillLocal) ok = ok && (n < d.n_sink || n > pos - d.window);
            if (MODE == kPrefillSparse) ok = (member >> (nt * 4 + e)) & 1u;
            if (!ok) s[nt][e] = -INFINITY;
          }
        }
      }
      // ---- online softmax ----
      float ta = -INFINITY, tb = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        ta = fmaxf(ta, fmaxf(s[nt][0], s[nt][1]));
        tb = fmaxf(tb, fmaxf(s[nt][2], s[nt][3]));
      }
      ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, 1));
      ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, 2));
      tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, 1));
      tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, 2));
      const float na = fmaxf(mx_a, ta * sc2), nb = fmaxf(mx_b, tb * sc2);
      const float ca = (na == -INFINITY) ? 1.f : fast_ex2(mx_a - na);
      const float cb = (nb == -INFINITY) ? 1.f : fast_ex2(mx_b - nb);
      const float ba = (na == -INFINITY) ? 0.f : na, bb = (nb == -INFINITY) ? 0.f : nb;
      mx_a = na;
      mx_b = nb;
      float ra = 0.f, rb = 0.f;
      uint32_t pf[4][4];   // P as bf16 A fragments, one per 16 keys
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p0 = fast_ex2(s[nt][0] * sc2 - ba), p1 = fast_ex2(s[nt][1] * sc2 - ba);
        const float p2 = fast_ex2(s[nt][2] * sc2 - bb), p3 = fast_ex2(s[nt][3] * sc2 - bb);
        ra += p0 + p1;
        rb += p2 + p3;
        pf[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
        pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l_a = l_a * ca + ra;
      l_b = l_b * cb + rb;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        o[i][0] *= ca;
        o[i][1] *= ca;
        o[i][2] *= cb;
        o[i][3] *= cb;
      }
      // ---- O += P V ----
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {      // 16 keys per step
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {    // pairs of n8 tiles over the 128 dims
          uint32_t b[4];
          const int row = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int ch = dp * 2 + (lane >> 4);
          ldmatrix_x4_trans(b, v_u32 + swz(row, ch));
          mma_bf16_16816(o[2 * dp], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b[0], b[1], o[2 * dp]);
          mma_bf16_16816(o[2 * dp + 1], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b[2], b[3], o[2 * dp + 1]);
        }
      }
    }
    __syncthreads();   // the stage is refilled by the next iteration's prefetch
  }
  cp_async_wait<0>();

  // ---- epilogue ----
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
  const float ia = l_a > 0.f ? 1.f / l_a : 0.f, ib = l_b > 0.f ? 1.f / l_b : 0.f;
  if (row_a_ok) {
    __nv_bfloat16* dst = out + ((int64_t)(r0 + pofs + g) * d.n_q + qh) * kHeadDim;
#pragma unroll
    for (int i = 0; i < 16; ++i)
      *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * c) = pack_bf16(o[i][0] * ia, o[i][1] * ia);
    if (lse && c == 0) lse[(int64_t)(r0 + pofs + g) * d.n_q + qh] = l_a > 0.f ? (mx_a + log2f(l_a)) * kLn2P : -INFINITY;
  }
  if (row_b_ok) {
    __nv_bfloat16* dst = out + ((int64_t)(r0 + pofs + g + 8) * d.n_q + qh) * kHeadDim;
#pragma unroll
    for (int i = 0; i < 16; ++i)
      *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * c) = pack_bf16(o[i][2] * ib, o[i][3] * ib);
    if (lse && c == 0) lse[(int64_t)(r0 + pofs + g + 8) * d.n_q + qh] = l_b > 0.f ? (mx_b + log2f(l_b)) * kLn2P : -INFINITY;
  }
}

template <int G, int MODE>
cudaError_t launch_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q,
                         const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start, int64_t C,
                         const float* sel_thresh, const int32_t* sel_tie_last, __nv_bfloat16* out, float* lse,
                         int n_units, cudaStream_t st) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(attn_prefill_kernel<G, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  constexpr int BMP = kRows / G;
  const int n_row_tiles = (int)((C + BMP - 1) / BMP);
  dim3 grid(n_row_tiles, n_units);
  attn_prefill_kernel<G, MODE><<<grid, kThreadsP, kSmemBytes, st>>>(cv, d, hm, q, qt, seq_id, q_start, (int)C,
                                                                    sel_thresh, sel_tie_last, out, lse, n_row_tiles);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t launch_mode(const CacheView& cv, const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q,
                        const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start, int64_t C, const float* sel_thresh,
                        const int32_t* sel_tie_last, __nv_bfloat16* out, float* lse, int n_units, cudaStream_t st) {
  switch (d.group) {
    case 1: return launch_typed<1, MODE>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse, n_units, st);
    case 2: return launch_typed<2, MODE>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse, n_units, st);
    case 4: return launch_typed<4, MODE>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse, n_units, st);
    case 8: return launch_typed<8, MODE>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse, n_units, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace

cudaError_t launch_attn_prefill(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                const __nv_bfloat16* q, const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start,
                                int64_t C, const float* sel_thresh, const int32_t* sel_tie_last,
                                __nv_bfloat16* out, float* lse, int32_t* status, int sm_count, cudaStream_t st) {
  (void)sm_count;
  if (C == 0) return cudaSuccess;
  // every mode runs on tcgen05 / TMEM / TMA; RTP_PREFILL_TC=0 selects the warp-MMA kernel of this file
  static const bool use_tc = [] { const char* e = getenv("RTP_PREFILL_TC"); return !(e && e[0] == '0'); }();
  if (mode == kPrefillSparse) {
    // one CTA column per index head; every query head of its KV head must be a retrieval head on it
    for (int j = 0; j < d.n_ih; ++j)
      if (hm.ih_nheads[j] != d.group) return cudaErrorNotSupported;
    for (int i = 0; i < d.n_ret; ++i)
      if (hm.ret_q_head[i] != hm.ih_kv[hm.q2ih[i]] * d.group + hm.slot_in_ih[i]) return cudaErrorNotSupported;
    if (use_tc)
      return launch_attn_prefill_tc(cv, d, hm, mode, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, st);
    return launch_mode<kPrefillSparse>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse,
                                       d.n_ih, st);
  }
  if (hm.n_kv_list == 0) return cudaSuccess;
  if (use_tc)
    return launch_attn_prefill_tc(cv, d, hm, mode, q, nullptr, nullptr, nullptr, seq_id, q_start, C, out, lse, status, st);
  if (mode == kPrefillLocal)
    return launch_mode<kPrefillLocal>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse,
                                      hm.n_kv_list, st);
  return launch_mode<kPrefillDense>(cv, d, hm, q, qt, seq_id, q_start, C, sel_thresh, sel_tie_last, out, lse,
                                    hm.n_kv_list, st);
}

}  // namespace rtp
