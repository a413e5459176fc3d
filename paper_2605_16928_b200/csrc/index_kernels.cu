// S0/S1: low-rank projections (Eq. 4 factors W^K k_pre and W^Q q_pre); S2/S3: materialised
// indexer scores with the softmax normaliser.
#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kProjTokens = 16;   // tokens (rows) per CTA
constexpr int kProjThreads = kProjTokens * kIndexDim;

// One CTA projects 16 rows of one projection head: thread (t, j) owns output j of row t and
// accumulates the 128 products in fp32 in channel order.
template <bool kKeys>
__global__ void __launch_bounds__(kProjThreads) project_kernel(
    CacheView cv, Dims d, HeadMaps hm, const __nv_bfloat16* __restrict__ src,
    const __nv_bfloat16* __restrict__ w, const int32_t* __restrict__ tok_seq,
    const int32_t* __restrict__ tok_pos, int64_t T, __nv_bfloat16* __restrict__ qt) {
  chain_wait();
  __shared__ float ws[kHeadDim * kIndexDim];                      // 8 KB
  __shared__ __align__(16) __nv_bfloat16 xs[kProjTokens][kHeadDim];  // 4 KB
  const int head = blockIdx.y;
  const int tid = threadIdx.x;
  const int64_t t0 = (int64_t)blockIdx.x * kProjTokens;

  {  // weights: 2048 bf16, 8 per thread
    const uint4 v = ld_nc_v4(w + (int64_t)head * kHeadDim * kIndexDim + tid * 8);
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(p[i]);
      ws[tid * 8 + 2 * i] = f.x;
      ws[tid * 8 + 2 * i + 1] = f.y;
    }
  }
  {  // rows: 16 x 256 B, one 16-byte load per thread
    const int r = tid >> 4, c = tid & 15;
    const int64_t t = t0 + r;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (t < T) {
      const int64_t row = kKeys ? (t * d.n_ih + head) : (t * d.n_q + hm.ret_q_head[head]);
      v = ld_stream_v4(src + row * kHeadDim + c * 8);
    }
    *reinterpret_cast<uint4*>(&xs[r][c * 8]) = v;
  }
  __syncthreads();

  const int r = tid >> 4, j = tid & 15;
  const int64_t t = t0 + r;
  float acc = 0.f;
#pragma unroll 16
  for (int c = 0; c < kHeadDim; ++c) acc = fmaf(__bfloat162float(xs[r][c]), ws[c * kIndexDim + j], acc);
  if (t >= T) return;
  const __nv_bfloat16 o = __float2bfloat16_rn(acc);
  if (kKeys) {
    const int seq = tok_seq[t], pos = tok_pos[t];
    if (seq < 0 || seq >= cv.batch || pos < 0 || (pos >> kPageShift) >= cv.max_pages) return;
    const int phys = cv.block_table[(int64_t)seq * cv.max_pages + (pos >> kPageShift)];
    if (phys < 0 || phys >= cv.num_pages) return;
    const int64_t at = (((int64_t)phys * cv.n_ih + head) * kPage + (pos & (kPage - 1))) * kIndexDim + j;
    if (cv.ikey_fp8)   // the fp32 sum straight to E4M3: nearest, ties to even, saturating at 448
      reinterpret_cast<uint8_t*>(cv.ikey)[at] = (uint8_t)__nv_cvt_float_to_fp8(acc, __NV_SATFINITE, __NV_E4M3);
    else
      cv.ikey[at] = o;
  } else {
    qt[(t * d.n_ret + head) * kIndexDim + j] = o;
  }
}

// ---- K/V append: one 16-byte chunk per thread, K and V -----------------------------------------
// k_new / v_new hold all n_src_heads KV heads of every token; the view stores those with a slot in its pool.
__global__ void kv_append_kernel(CacheView cv, const int n_src_heads, const __nv_bfloat16* __restrict__ k_new,
                                 const __nv_bfloat16* __restrict__ v_new, const int32_t* __restrict__ tok_seq,
                                 const int32_t* __restrict__ tok_pos, int64_t T, int32_t* status) {
  const int64_t chunks_per_tok = (int64_t)n_src_heads * 16;
  const int64_t total = T * chunks_per_tok;
  __nv_bfloat16* kp = const_cast<__nv_bfloat16*>(cv.k);
  __nv_bfloat16* vp = const_cast<__nv_bfloat16*>(cv.v);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = i / chunks_per_tok;
    const int rem = (int)(i % chunks_per_tok);
    const int head = rem >> 4, ch = rem & 15;
    const int slot = cv.kv_slot[head];
    if (slot == 0xff) continue;   // the head lives in the other pool
    const int seq = tok_seq[t], pos = tok_pos[t];
    if (seq < 0 || seq >= cv.batch || pos < 0 || pos >= cv.cap_tokens) {
      set_status(status, RTP_ERR_INVALID);
      continue;
    }
    const int phys = cv.block_table[(int64_t)seq * cv.max_pages + page_entry(cv, pos >> kPageShift)];
    if (phys < 0 || phys >= cv.num_pages) {
      set_status(status, RTP_ERR_INVALID);
      continue;
    }
    const int64_t src = (t * n_src_heads + head) * kHeadDim + ch * 8;
    const int64_t dst = (((int64_t)phys * cv.n_kv + slot) * kPage + (pos & (kPage - 1))) * kHeadDim + ch * 8;
    *reinterpret_cast<uint4*>(kp + dst) = ld_stream_v4(k_new + src);
    *reinterpret_cast<uint4*>(vp + dst) = ld_stream_v4(v_new + src);
  }
}

// ---- materialised scores -----------------------------------------------------------------------
constexpr int kScoreWarps = 4;

// grid = (R * n_ih, splits).  Each CTA scans a contiguous range of pages of one (row, index head)
// for all retrieval heads attached to that index head.
template <bool F8>
__global__ void __launch_bounds__(kScoreWarps * 32) score_kernel(
    CacheView cv, Dims d, HeadMaps hm, Rows rows, const __nv_bfloat16* __restrict__ qt,
    float* __restrict__ scores, int64_t score_stride, float2* __restrict__ partial, int n_splits,
    int32_t* status) {
  const int64_t r = blockIdx.x / d.n_ih;
  const int ih = blockIdx.x % d.n_ih;
  const int split = blockIdx.y;
  const int nh = hm.ih_nheads[ih];
  if (nh == 0) return;
  const int seq = rows.row_seq(r);
  int n_keys = rows.row_pos(r) + 1;
  {
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;   // (never beyond the block table)
    if (n_keys > sl) {
      if (threadIdx.x == 0) set_status(status, RTP_ERR_INVALID);
      n_keys = sl;
    }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, c = lane & 3;
  const int n_pages = (n_keys + kPage - 1) >> kPageShift;
  const int per = (n_pages + n_splits - 1) / n_splits;
  const int p_lo = split * per;
  const int p_hi = min(n_pages, p_lo + per);

  QFrag qf = load_qfrag(qt + r * d.n_ret * kIndexDim, hm.ih_heads[ih], nh, lane);
  if (F8 && !qfrag_to_f16(qf)) set_status(status, RTP_ERR_UNSUPPORTED);   // a projected query beyond fp16's range
  const int head_lo = g < nh ? hm.ih_heads[ih][g] : -1;
  const int head_hi = g + 8 < nh ? hm.ih_heads[ih][g + 8] : -1;
  float m_lo = -INFINITY, l_lo = 0.f, m_hi = -INFINITY, l_hi = 0.f;

  for (int p = p_lo + warp; p < p_hi; p += kScoreWarps) {
    uint4 v[4];
    uint2 v8[4];
    if (F8) {
      const uint8_t* base = ikey_page_ptr8(cv, seq, p, ih);
#pragma unroll
      for (int i = 0; i < 4; ++i) v8[i] = ld_stream_v2(base + (i * 32 + lane) * 8);
    } else {
      const __nv_bfloat16* base = ikey_page_ptr(cv, seq, p, ih);
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] = ld_stream_v4(base + (i * 32 + lane) * 8);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s_lo[4], s_hi[4];
      if (F8) score16_f8(qf, v8[i], lane, s_lo, s_hi); else score16(qf, v[i], lane, s_lo, s_hi);
      const int n0 = p * kPage + i * 16 + 4 * c;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int n = n0 + e;
        if (n >= n_keys) continue;
        if (head_lo >= 0) {
          const float s = finish_score(s_lo[e], d.score_scale);
          if (scores) scores[(r * d.n_ret + head_lo) * score_stride + n] = s;
          const float mn = fmaxf(m_lo, s);
          l_lo = l_lo * __expf(m_lo - mn) + __expf(s - mn);
          m_lo = mn;
        }
        if (head_hi >= 0) {
          const float s = finish_score(s_hi[e], d.score_scale);
          if (scores) scores[(r * d.n_ret + head_hi) * score_stride + n] = s;
          const float mn = fmaxf(m_hi, s);
          l_hi = l_hi * __expf(m_hi - mn) + __expf(s - mn);
          m_hi = mn;
        }
      }
    }
  }
  // combine the four lanes of a group, then the warps through shared memory
  __shared__ float2 red[kScoreWarps][16];
#pragma unroll
  for (int o = 1; o <= 2; o <<= 1) {
    float mo = __shfl_xor_sync(0xffffffffu, m_lo, o), lo = __shfl_xor_sync(0xffffffffu, l_lo, o);
    float mn = fmaxf(m_lo, mo);
    l_lo = (mn == -INFINITY) ? 0.f : l_lo * __expf(m_lo - mn) + lo * __expf(mo - mn);
    m_lo = mn;
    mo = __shfl_xor_sync(0xffffffffu, m_hi, o), lo = __shfl_xor_sync(0xffffffffu, l_hi, o);
    mn = fmaxf(m_hi, mo);
    l_hi = (mn == -INFINITY) ? 0.f : l_hi * __expf(m_hi - mn) + lo * __expf(mo - mn);
    m_hi = mn;
  }
  if (c == 0) {
    red[warp][g] = make_float2(m_lo, l_lo);
    red[warp][g + 8] = make_float2(m_hi, l_hi);
  }
  __syncthreads();
  if (threadIdx.x < nh) {
    float m = -INFINITY, l = 0.f;
    for (int w = 0; w < kScoreWarps; ++w) {
      const float2 x = red[w][threadIdx.x];
      const float mn = fmaxf(m, x.x);
      if (mn != -INFINITY) l = l * __expf(m - mn) + x.y * __expf(x.x - mn);
      m = mn;
    }
    const int head = hm.ih_heads[ih][threadIdx.x];
    partial[(r * d.n_ret + head) * n_splits + split] = make_float2(m, l);
  }
}

__global__ void score_merge_kernel(const float2* __restrict__ partial, int n_splits, int64_t n_rowheads,
                                   float* __restrict__ row_max, float* __restrict__ row_sum) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_rowheads) return;
  float m = -INFINITY, l = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float2 x = partial[i * n_splits + s];
    const float mn = fmaxf(m, x.x);
    if (mn != -INFINITY) l = l * __expf(m - mn) + x.y * __expf(x.x - mn);
    m = mn;
  }
  if (row_max) row_max[i] = m;
  if (row_sum) row_sum[i] = l;
}

int score_splits(const Dims& d, int64_t R, int64_t max_len, int sm_count) {
  const int64_t pages = (max_len + kPage - 1) / kPage;
  int64_t want = (4LL * sm_count + R * d.n_ih - 1) / (R * d.n_ih);
  int64_t cap = (pages + 31) / 32;   // at least 32 pages (2048 keys) per CTA
  int64_t s = want < cap ? want : cap;
  if (s < 1) s = 1;
  if (s > 1024) s = 1024;
  return (int)s;
}

}  // namespace

cudaError_t launch_kv_append(const CacheView& cv, int n_src_heads, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new,
                             const int32_t* tok_seq, const int32_t* tok_pos, int64_t T, int32_t* status,
                             cudaStream_t st) {
  if (T == 0) return cudaSuccess;
  const int64_t total = T * n_src_heads * 16;
  int64_t blocks = (total + 255) / 256;
  const int64_t cap = (int64_t)current_sm_count(148) * 16;   // a few waves of grid-stride blocks
  if (blocks > cap) blocks = cap;
  kv_append_kernel<<<(unsigned)blocks, 256, 0, st>>>(cv, n_src_heads, k_new, v_new, tok_seq, tok_pos, T, status);
  return cudaGetLastError();
}

cudaError_t launch_index_keys(const CacheView& cv, const Dims& d, const __nv_bfloat16* k_pre,
                              const __nv_bfloat16* w_k, const int32_t* tok_seq, const int32_t* tok_pos,
                              int64_t T, cudaStream_t st) {
  if (T == 0) return cudaSuccess;
  HeadMaps hm = {};
  dim3 grid((unsigned)((T + kProjTokens - 1) / kProjTokens), d.n_ih);
  (void)launch_chained(project_kernel<true>, dim3(grid), dim3(kProjThreads), 0, st, cv, d, hm, k_pre, w_k, tok_seq, tok_pos, T, nullptr);
  return cudaGetLastError();
}

cudaError_t launch_index_queries(const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q_pre,
                                 const __nv_bfloat16* w_q, int64_t R, __nv_bfloat16* qt, cudaStream_t st) {
  if (R == 0 || d.n_ret == 0) return cudaSuccess;
  CacheView cv = {};
  dim3 grid((unsigned)((R + kProjTokens - 1) / kProjTokens), d.n_ret);
  (void)launch_chained(project_kernel<false>, dim3(grid), dim3(kProjThreads), 0, st, cv, d, hm, q_pre, w_q, nullptr, nullptr, R, qt);
  return cudaGetLastError();
}

size_t score_workspace_bytes(const Dims& d, int64_t R, int64_t max_len, int sm_count) {
  if (R <= 0) return 0;
  return (size_t)R * d.n_ret * score_splits(d, R, max_len, sm_count) * sizeof(float2);
}

cudaError_t launch_index_score(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const __nv_bfloat16* qt, int64_t max_len, float* scores, int64_t score_stride,
                               float* row_max, float* row_sum, void* ws, int32_t* status, int sm_count,
                               cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  const int n_splits = score_splits(d, rows.R, max_len, sm_count);
  dim3 grid((unsigned)(rows.R * d.n_ih), n_splits);
  if (cv.ikey_fp8)
    score_kernel<true><<<grid, kScoreWarps * 32, 0, st>>>(cv, d, hm, rows, qt, scores, score_stride,
                                                          reinterpret_cast<float2*>(ws), n_splits, status);
  else
    score_kernel<false><<<grid, kScoreWarps * 32, 0, st>>>(cv, d, hm, rows, qt, scores, score_stride,
                                                           reinterpret_cast<float2*>(ws), n_splits, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (row_max || row_sum) {
    const int64_t n = rows.R * d.n_ret;
    score_merge_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(reinterpret_cast<const float2*>(ws),
                                                                     n_splits, n, row_max, row_sum);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace rtp
