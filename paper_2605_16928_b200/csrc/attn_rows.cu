// S5 / S7 (decode) / S8 / S9 (decode): attention of single query rows over a token set (Eq. 5):
// a selection list, the sink + window pattern, or the full causal prefix.  Bandwidth-bound, so the kernel is built
// around keeping many K / V rows in flight with few instructions per row:
//   - the set is split over CTAs (merged by log-sum-exp) and, inside a CTA, dealt to four warps in tiles of 16 tokens;
//   - every warp owns a ring of three tiles in shared memory, filled with 16-byte cp.async copies (a half-warp per
//     256-byte row) two tiles ahead of the one it works on; where a row lives (list entry -> block table -> offset) is
//     resolved another two tiles ahead, so that none of these dependent loads is waited for;
//   - Q K^T and P V of a tile are warp MMAs (m16n8k16, bf16 -> fp32): the G query heads of the KV group are rows of the
//     A operand (the other rows are zero), the tile's K rows are read with ldmatrix, its V rows with ldmatrix.trans,
//     from a layout whose 16-byte chunks are XOR-swizzled with the token number (no bank conflicts).
#include <mutex>

#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kTileTok = 16;                               // tokens per tile
constexpr int kRing = 3;                                   // tiles per warp in shared memory
constexpr int kTileBytes = kTileTok * kHeadDim * 2;        // K (or V) rows of a tile: 4 KB
constexpr int kWarpRingBytes = kRing * 2 * kTileBytes;     // 24 KB
constexpr int kRowsSmem = kWarps * kWarpRingBytes;         // 96 KB: two CTAs per SM
constexpr int kPartial = kHeadDim + 2;                     // acc[128], m, l
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void cp16z(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// d (rows g of the 16 x 8 result) += A B, where rows 8-15 of A are zero: only the two accumulators of row g are kept.
__device__ __forceinline__ void mma_row8(float (&d)[2], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "{\n"
      ".reg .f32 x2, x3;\n"
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,x2,x3}, {%2,%3,%4,%3}, {%5,%6}, {%0,%1,%7,%7};\n"
      "}\n"
      : "+f"(d[0]), "+f"(d[1])
      : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1), "f"(0.f));
}
// byte offset of 16-byte chunk ch (0..15) of token t inside a tile
__device__ __forceinline__ uint32_t tile_off(int t, int ch) { return (uint32_t)(t * 256 + (((ch & 8) | ((ch ^ t) & 7)) << 4)); }

template <int G, int SET>
__global__ void __launch_bounds__(kThreads, 2) attn_rows_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows, const int n_units,
    const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ sel_idx, const int64_t sel_stride,
    const int32_t* __restrict__ sel_count, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
    float* __restrict__ partial, const int n_splits, int32_t* status) {
  chain_wait();
  static_assert(G >= 1 && G <= 8, "the query heads of a KV group are rows 0..7 of the MMA");
  extern __shared__ __align__(128) unsigned char smem_rows[];

  const int64_t r = blockIdx.x / n_units;
  const int u = blockIdx.x % n_units;
  const int split = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, c = lane & 3;

  int qh0, kvh;
  if (SET == kSetList || SET == kSetPages) {
    qh0 = hm.ret_q_head[u];
    kvh = qh0 / d.group;
  } else {
    kvh = hm.kv_list[u];
    qh0 = kvh * d.group;
  }
  const int seq = rows.row_seq(r);
  const int m_pos = rows.row_pos(r);
  int n_keys = m_pos + 1;
  {
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.cap_tokens) : 0;   // (never beyond the block table)
    if (n_keys > sl) {
      if (threadIdx.x == 0) set_status(status, RTP_ERR_INVALID);
      n_keys = sl;
    }
    if (n_keys < 0) n_keys = 0;
  }
  // enumerate the set as t = 0 .. n_set-1
  int n_set, ns = 0, wlo = 0;
  const int32_t* ids = nullptr;
  if (SET == kSetList || SET == kSetPages) {
    const int64_t rh = r * d.n_ret + u;
    n_set = min((int64_t)sel_count[rh], sel_stride);
    n_set = max(n_set, 0);
    if (SET == kSetPages) n_set *= kPage;   // every listed page is 64 entries (the row's last page: fewer are causal)
    ids = sel_idx + rh * sel_stride;
  } else if (SET == kSetUnion) {
    const int64_t ru = r * n_units + u;
    n_set = max(min((int64_t)sel_count[ru], sel_stride), (int64_t)0) * kPage;
    ids = sel_idx + ru * sel_stride;
  } else if (SET == kSetLocal) {
    ns = min(d.n_sink, n_keys);
    wlo = max(ns, n_keys - d.window);
    n_set = ns + max(0, n_keys - wlo);
  } else {
    n_set = n_keys;
  }
  // (a union list is cut at page boundaries: the head flags of a 16-token tile are then those of one entry)
  const int per = SET == kSetUnion ? (((n_set >> kPageShift) + n_splits - 1) / n_splits) << kPageShift
                                   : (n_set + n_splits - 1) / n_splits;
  const int t_lo = split * per;
  const int t_hi = min(n_set, t_lo + per);
  const int n_tiles = t_hi > t_lo ? (t_hi - t_lo + kTileTok - 1) / kTileTok : 0;
  const int n_mine = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;   // tiles warp, warp + 4, ...

  // A fragments of the queries: row g = head g of the group (zero rows beyond G), 8 steps of 16 dims
  uint32_t qa[8][2];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    qa[ks][0] = 0u;
    qa[ks][1] = 0u;
    if (g < G) {
      const __nv_bfloat16* qp = q + ((int64_t)r * d.n_q + qh0 + g) * kHeadDim + 16 * ks + 2 * c;
      qa[ks][0] = *reinterpret_cast<const uint32_t*>(qp);
      qa[ks][1] = *reinterpret_cast<const uint32_t*>(qp + 8);
    }
  }
  const float sc = d.sm_scale * kLog2e;   // logits in log2 units
  float o[16][2];                         // row g, dims 8 j + 2 c, + 1
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = 0.f;
  float m_run = -INFINITY, l_part = 0.f;

  const int64_t bt_base = (int64_t)seq * cv.max_pages;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem_rows) + warp * kWarpRingBytes;
  // Token of entry (lane & 15) of this warp's i-th tile, or -1, and the physical page it lives in.  The loads and the
  // checks of what they return are separate steps: a value is looked at one tile later than it was requested, so that
  // the warp never waits for these dependent loads.
  auto raw_tok = [&](int i) -> int {
    const int t = t_lo + (warp + i * kWarps) * kTileTok + (lane & 15);
    if (i >= n_mine || t >= t_hi) return -1;
    if (SET == kSetList) return __ldg(ids + t);
    if (SET == kSetPages) return __ldg(ids + (t >> kPageShift)) * kPage + (t & (kPage - 1));
    if (SET == kSetUnion) return (__ldg(ids + (t >> kPageShift)) & 0xffffff) * kPage + (t & (kPage - 1));
    if (SET == kSetLocal) return t < ns ? t : wlo + (t - ns);
    return t;
  };
  auto check_tok = [&](int tok) -> int {
    if (SET == kSetList && tok != -1 && (tok < 0 || tok >= n_keys)) {
      set_status(status, RTP_ERR_INVALID);
      return -1;
    }
    if ((SET == kSetPages || SET == kSetUnion) && tok != -1) {
      // a listed page must hold a causal key; the positions of the row's last page beyond its own are left out quietly
      if (tok < 0 || (tok >> kPageShift) > ((n_keys - 1) >> kPageShift) || n_keys == 0) {
        set_status(status, RTP_ERR_INVALID);
        return -1;
      }
      if (tok >= n_keys) return -1;
    }
    return tok;
  };
  const int kslot = cv.kv_slot[kvh];   // the KV head's place inside a page of this pool
  auto raw_phys = [&](int tok) -> int { return tok >= 0 ? __ldg(cv.block_table + bt_base + page_entry(cv, tok >> kPageShift)) : 0; };
  auto check_phys = [&](int phys) -> int {
    if ((unsigned)phys < (unsigned)cv.num_pages) return phys;
    set_status(status, RTP_ERR_INVALID);
    return 0;
  };
  // requests the K and V rows of a tile: token tt of the tile is copied by the half-warp (tt & 1) in step tt >> 1
  auto issue = [&](int stage, int tok, int phys) {
    const int64_t off = (((int64_t)phys * cv.n_kv + kslot) * kPage + (tok & (kPage - 1))) * kHeadDim;
    const uint32_t sk = ring + stage * 2 * kTileBytes, sv = sk + kTileBytes;
    const int ch = lane & 15;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int tt = 2 * i + (lane >> 4);
      const int64_t o_t = __shfl_sync(0xffffffffu, off, tt);
      const bool ok = __shfl_sync(0xffffffffu, tok, tt) >= 0;
      const int64_t src = ok ? o_t + ch * 8 : 0;
      cp16z(sk + tile_off(tt, ch), cv.k + src, ok);
      cp16z(sv + tile_off(tt, ch), cv.v + src, ok);
    }
  };
  // prologue: two tiles requested; the addresses of the third resolved, the tokens of the fourth on their way
  int tok_c[kRing];   // tokens of the tiles in the ring (for the validity mask)
  {
    const int t0 = check_tok(raw_tok(0)), t1 = check_tok(raw_tok(1));
    const int p0 = check_phys(raw_phys(t0)), p1 = check_phys(raw_phys(t1));
    issue(0, t0, p0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    issue(1, t1, p1);
    asm volatile("cp.async.commit_group;" ::: "memory");
    tok_c[0] = t0;
    tok_c[1] = t1;
    tok_c[2] = -1;
  }
  int tok_a = check_tok(raw_tok(2));
  int phys_a = raw_phys(tok_a);   // (looked at when tile 2 is requested)
  int tok_b = raw_tok(3);         // (looked at one step later)

#pragma unroll 1
  for (int i0 = 0; i0 < n_mine; i0 += kRing) {
#pragma unroll
    for (int sgi = 0; sgi < kRing; ++sgi) {
      const int i = i0 + sgi;
      if (i < n_mine) {   // uniform in the warp
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncwarp();
        // tile i + 2 goes where tile i - 1 was
        const int next_stage = (sgi + 2) % kRing;
        issue(next_stage, tok_a, check_phys(phys_a));
        asm volatile("cp.async.commit_group;" ::: "memory");
        tok_c[next_stage] = tok_a;
        tok_a = check_tok(tok_b);       // (requested one step ago)
        phys_a = raw_phys(tok_a);       // looked at in the next step
        tok_b = raw_tok(i + 4);         // looked at in the next step, used in the one after

        const uint32_t sk = ring + sgi * 2 * kTileBytes, sv = sk + kTileBytes;
        const uint32_t vmask = __ballot_sync(0xffffffffu, tok_c[sgi] >= 0) & 0xffffu;   // bit t = token t of the tile exists
        // union lists: which query heads of the group selected the page of this tile (the entry was loaded when the
        // tile was requested: it comes from the L1 cache)
        bool head_on = true;
        if (SET == kSetUnion) {
          const int t_first = t_lo + (warp + i * kWarps) * kTileTok;
          head_on = ((uint32_t)__ldg(ids + (t_first >> kPageShift)) >> (24 + g)) & 1u;
        }
        // ---- S = Q K^T: two 8-token halves ----
        float s[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        {
          const int mi = lane >> 3, rr = lane & 7;
          const int tk = (mi >> 1) * 8 + rr;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t b[4];
            ldsm4(sk + tile_off(tk, 2 * ks + (mi & 1)), b);
            mma_row8(s[0], qa[ks][0], qa[ks][1], b[0], b[1]);
            mma_row8(s[1], qa[ks][0], qa[ks][1], b[2], b[3]);
          }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const bool ok = ((vmask >> (8 * nt + 2 * c + e)) & 1u) && head_on;
            s[nt][e] = ok ? s[nt][e] * sc : -INFINITY;
            mx = fmaxf(mx, s[nt][e]);
          }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        if (__any_sync(0xffffffffu, m_new > m_run)) {
          const float corr = (m_run == -INFINITY) ? 0.f : fast_ex2(m_run - m_new);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            o[j][0] *= corr;
            o[j][1] *= corr;
          }
          l_part *= corr;
          m_run = m_new;
        }
        const float mb = (m_run == -INFINITY) ? 0.f : m_run;
        const float p00 = fast_ex2(s[0][0] - mb), p01 = fast_ex2(s[0][1] - mb);
        const float p10 = fast_ex2(s[1][0] - mb), p11 = fast_ex2(s[1][1] - mb);
        l_part += (p00 + p01) + (p10 + p11);
        uint32_t pa0, pa2;
        {
          const __nv_bfloat162 x = __floats2bfloat162_rn(p00, p01), y = __floats2bfloat162_rn(p10, p11);
          pa0 = *reinterpret_cast<const uint32_t*>(&x);
          pa2 = *reinterpret_cast<const uint32_t*>(&y);
        }
        // ---- O += P V: 16 slices of eight dims, two per ldmatrix ----
        {
          const int mi = lane >> 3, rr = lane & 7;
          const int tk = (mi & 1) * 8 + rr;
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            uint32_t b[4];
            ldsm4t(sv + tile_off(tk, j + (mi >> 1)), b);
            mma_row8(o[j], pa0, pa2, b[0], b[1]);
            mma_row8(o[j + 1], pa0, pa2, b[2], b[3]);
          }
        }
      }
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();   // the rings are free: they now hold the warps' partial results

  float l_run = l_part;
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  float* red = reinterpret_cast<float*>(smem_rows);   // [kWarps][G][kPartial]
  if (g < G) {
    float* rw = red + (warp * G + g) * kPartial;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      rw[8 * j + 2 * c] = o[j][0];
      rw[8 * j + 2 * c + 1] = o[j][1];
    }
    if (c == 0) {
      rw[kHeadDim] = m_run;
      rw[kHeadDim + 1] = l_run;
    }
  }
  __syncthreads();
  const int dim = threadIdx.x;  // 128 threads = 128 dims
#pragma unroll
  for (int gg = 0; gg < G; ++gg) {
    float mt = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) mt = fmaxf(mt, red[(w * G + gg) * kPartial + kHeadDim]);
    float lt = 0.f, a = 0.f;
    if (mt != -INFINITY) {
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float* rw = red + (w * G + gg) * kPartial;
        const float wgt = fast_ex2(rw[kHeadDim] - mt);
        lt += rw[kHeadDim + 1] * wgt;
        a += rw[dim] * wgt;
      }
    }
    const int64_t oh = (int64_t)r * d.n_q + qh0 + gg;
    // (a retrieval head inside a local group is not a local call's; a local head inside a retrieval group not a union call's)
    if ((SET == kSetLocal || SET == kSetUnion) && hm.skips(qh0 + gg)) continue;
    if (n_splits == 1) {
      out[oh * kHeadDim + dim] = __float2bfloat16_rn(lt > 0.f ? a / lt : 0.f);
      if (lse && dim == 0) lse[oh] = lt > 0.f ? (mt + log2f(lt)) * kLn2 : -INFINITY;
    } else {
      float* p = partial + (((int64_t)blockIdx.x * G + gg) * n_splits + split) * kPartial;
      p[dim] = a;
      if (dim == 0) {
        p[kHeadDim] = mt;
        p[kHeadDim + 1] = lt;
      }
    }
  }
}

// One CTA per (unit, head of the group): log-sum-exp merge of the split partials.
template <int SET>
__global__ void __launch_bounds__(kHeadDim) attn_merge_kernel(const Dims d, const HeadMaps hm, const int n_units,
                                                              const int G, const float* __restrict__ partial,
                                                              const int n_splits, __nv_bfloat16* __restrict__ out,
                                                              float* __restrict__ lse) {
  chain_wait();
  const int64_t unit = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t r = unit / n_units;
  const int u = unit % n_units;
  const int qh = (SET == kSetList || SET == kSetPages) ? hm.ret_q_head[u] : hm.kv_list[u] * d.group + g;
  if ((SET == kSetLocal || SET == kSetUnion) && hm.skips(qh)) return;
  const float* p = partial + ((unit * G + g) * (int64_t)n_splits) * kPartial;
  const int dim = threadIdx.x;
  float mt = -INFINITY;
  for (int s = 0; s < n_splits; ++s) mt = fmaxf(mt, p[(int64_t)s * kPartial + kHeadDim]);
  float lt = 0.f, a = 0.f;
  if (mt != -INFINITY) {
    for (int s = 0; s < n_splits; ++s) {
      const float w = fast_ex2(p[(int64_t)s * kPartial + kHeadDim] - mt);
      lt += p[(int64_t)s * kPartial + kHeadDim + 1] * w;
      a += p[(int64_t)s * kPartial + dim] * w;
    }
  }
  const int64_t oh = r * d.n_q + qh;
  out[oh * kHeadDim + dim] = __float2bfloat16_rn(lt > 0.f ? a / lt : 0.f);
  if (lse && dim == 0) lse[oh] = lt > 0.f ? (mt + log2f(lt)) * kLn2 : -INFINITY;
}

// Split count of a call.  Long contiguous sets (dense, sink + window) get at most two full rounds of two resident
// CTAs per SM, rounded down: a few CTAs beyond a full round would cost a round of their own (dense decode at
// B = 4 / 512K: 1411 -> 1246 us).  List gathers are short and latency-bound, their count is rounded up.
int plan_splits(int64_t units, int64_t max_set, int sm_count, bool round_up) {
  if (units <= 0) return 1;
  int64_t want = (4LL * sm_count + (round_up ? units - 1 : 0)) / units;
  int64_t cap = (max_set + 511) / 512;                   // at least 512 tokens (eight tiles per warp) per CTA
  int64_t s = want < cap ? want : cap;
  if (s < 1) s = 1;
  if (s > 512) s = 512;
  return (int)s;
}

int64_t max_set_len(const Dims& d, int set, int64_t sel_stride, int64_t max_len) {
  if (set == kSetList) return sel_stride < max_len ? sel_stride : max_len;
  if (set == kSetPages || set == kSetUnion) return sel_stride * kPage < max_len ? sel_stride * kPage : (max_len + kPage - 1) / kPage * kPage;
  if (set == kSetLocal) {
    const int64_t w = (int64_t)d.n_sink + d.window;
    return w < max_len ? w : max_len;
  }
  return max_len;
}

template <int G, int SET>
cudaError_t launch_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows, int n_units,
                         const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                         const int32_t* sel_count, __nv_bfloat16* out, float* lse, float* partial, int n_splits,
                         int32_t* status, cudaStream_t st) {
  dim3 grid((unsigned)(rows.R * n_units), n_splits);
  static PerDeviceOnce once;   // (one per instantiation)
  cudaError_t e = set_dyn_smem_once(attn_rows_kernel<G, SET>, kRowsSmem, once);
  if (e != cudaSuccess) return e;
  (void)launch_chained(attn_rows_kernel<G, SET>, dim3(grid), dim3(kThreads), kRowsSmem, st, cv, d, hm, rows, n_units, q, sel_idx, sel_stride,
                                                              sel_count, out, lse, partial, n_splits, status);
  e = cudaGetLastError();
  if (e != cudaSuccess || n_splits == 1) return e;
  (void)launch_chained(attn_merge_kernel<SET>, dim3((unsigned)(rows.R * n_units * G)), dim3(kHeadDim), 0, st, d, hm, n_units, G, partial,
                                                                                n_splits, out, lse);
  return cudaGetLastError();
}

}  // namespace

size_t attn_rows_workspace_bytes(const Dims& d, int64_t R, int n_units, int group, int sm_count, int64_t max_len) {
  if (R <= 0 || n_units <= 0) return 0;
  const int n_splits = plan_splits(R * n_units, max_len, sm_count, true);   // (the larger of the two roundings)
  return (size_t)R * n_units * group * n_splits * kPartial * sizeof(float);
}

cudaError_t launch_attn_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows, int set,
                             const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                             const int32_t* sel_count, __nv_bfloat16* out, float* lse, void* ws, size_t ws_bytes,
                             int64_t max_len, int32_t* status, int sm_count, cudaStream_t st) {
  const bool per_head = set == kSetList || set == kSetPages;   // one set per retrieval query head
  const int n_units = per_head ? d.n_ret : hm.n_kv_list;
  if (rows.R == 0 || n_units == 0) return cudaSuccess;
  const int G = per_head ? 1 : d.group;
  int n_splits = plan_splits(rows.R * n_units, max_set_len(d, set, sel_stride, max_len), sm_count, set == kSetList);
  // never plan more splits than the workspace holds
  const size_t per_split = (size_t)rows.R * n_units * G * kPartial * sizeof(float);
  if (n_splits > 1 && (size_t)n_splits * per_split > ws_bytes) n_splits = (int)(ws_bytes / per_split);
  if (n_splits < 1) n_splits = 1;
  float* partial = reinterpret_cast<float*>(ws);
#define RTP_LAUNCH(GG, SS)                                                                                   \
  return launch_typed<GG, SS>(cv, d, hm, rows, n_units, q, sel_idx, sel_stride, sel_count, out, lse, partial, \
                              n_splits, status, st)
  if (set == kSetList) RTP_LAUNCH(1, kSetList);
  if (set == kSetPages) RTP_LAUNCH(1, kSetPages);
  if (set == kSetUnion) {
    if (G == 1) RTP_LAUNCH(1, kSetUnion);
    if (G == 2) RTP_LAUNCH(2, kSetUnion);
    if (G == 4) RTP_LAUNCH(4, kSetUnion);
    if (G == 8) RTP_LAUNCH(8, kSetUnion);
  }
  if (set == kSetLocal) {
    if (G == 1) RTP_LAUNCH(1, kSetLocal);
    if (G == 2) RTP_LAUNCH(2, kSetLocal);
    if (G == 4) RTP_LAUNCH(4, kSetLocal);
    if (G == 8) RTP_LAUNCH(8, kSetLocal);
  } else {
    if (G == 1) RTP_LAUNCH(1, kSetDense);
    if (G == 2) RTP_LAUNCH(2, kSetDense);
    if (G == 4) RTP_LAUNCH(4, kSetDense);
    if (G == 8) RTP_LAUNCH(8, kSetDense);
  }
#undef RTP_LAUNCH
  return cudaErrorInvalidValue;
}

// ---- split partials in a static device array (entry point for callers that must not allocate) --------
// kStaticScratchBytes of global memory are part of the library image on every GPU that loads it.
constexpr size_t kStaticScratchBytes = 512u << 10;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device
}  // namespace

size_t attn_rows_static_scratch_bytes() { return kStaticScratchBytes; }

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can use: the
// device address is looked up once per device (with that device current) and cached.
cudaError_t launch_attn_rows_static(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                    const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                                    const int32_t* sel_count, __nv_bfloat16* out, float* lse, int64_t max_len,
                                    int32_t* status, int sm_count, size_t* needed_bytes, cudaStream_t st) {
  *needed_bytes = 0;
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  const int n_splits = plan_splits(rows.R * d.n_ret, max_set_len(d, kSetList, sel_stride, max_len), sm_count, true);
  const size_t need = n_splits > 1 ? (size_t)rows.R * d.n_ret * n_splits * kPartial * sizeof(float) : 0;
  *needed_bytes = need;
  if (need > kStaticScratchBytes) return cudaErrorMemoryAllocation;   // reported as RTP_ERR_CAPACITY by the caller
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  void* ptr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
      e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (e != cudaSuccess) return e;
      g_scratch_ptr[dev] = ptr;
    }
    ptr = g_scratch_ptr[dev];
  }
  return launch_typed<1, kSetList>(cv, d, hm, rows, d.n_ret, q, sel_idx, sel_stride, sel_count, out, lse,
                                   reinterpret_cast<float*>(ptr), n_splits, status, st);
}

}  // namespace rtp
