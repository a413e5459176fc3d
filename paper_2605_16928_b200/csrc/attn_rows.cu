// S5 / S7 (decode) / S8 / S9 (decode): attention of single query rows over a token set (Eq. 5):
// a selection list, the sink + window pattern, or the full causal prefix.  Bandwidth-bound: every
// K and V row is read once with 16-byte loads (a half-warp per 256-byte row), all query heads of a
// KV group share the loaded rows, the set is split over CTAs and merged by log-sum-exp.
#include <mutex>

#include "rtp_device.cuh"

namespace rtp {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kStreams = kWarps * 2;   // one online-softmax stream per half-warp
constexpr int kUnroll = 4;             // tokens in flight per half-warp
constexpr int kPartial = kHeadDim + 2; // acc[128], m, l
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 x = __bfloat1622float2(p[i]);
    f[2 * i] = x.x;
    f[2 * i + 1] = x.y;
  }
}

template <int G, int SET>
__global__ void __launch_bounds__(kThreads, (G == 1) ? 6 : 1) attn_rows_kernel(
    const CacheView cv, const Dims d, const HeadMaps hm, const Rows rows, const int n_units,
    const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ sel_idx, const int64_t sel_stride,
    const int32_t* __restrict__ sel_count, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
    float* __restrict__ partial, const int n_splits, int32_t* status) {
  __shared__ float red[kStreams][G][kPartial];

  const int64_t r = blockIdx.x / n_units;
  const int u = blockIdx.x % n_units;
  const int split = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int l16 = lane & 15, hw = lane >> 4;
  const int stream = warp * 2 + hw;

  int qh0, kvh;
  if (SET == kSetList) {
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
    const int sl = (seq >= 0 && seq < cv.batch) ? min(cv.seq_lens[seq], cv.max_pages * kPage) : 0;   // (never beyond the block table)
    if (n_keys > sl) {
      if (threadIdx.x == 0) set_status(status, RTP_ERR_INVALID);
      n_keys = sl;
    }
    if (n_keys < 0) n_keys = 0;
  }
  // enumerate the set as t = 0 .. n_set-1
  int n_set, ns = 0, wlo = 0;
  const int32_t* ids = nullptr;
  if (SET == kSetList) {
    const int64_t rh = r * d.n_ret + u;
    n_set = min((int64_t)sel_count[rh], sel_stride);
    n_set = max(n_set, 0);
    ids = sel_idx + rh * sel_stride;
  } else if (SET == kSetLocal) {
    ns = min(d.n_sink, n_keys);
    wlo = max(ns, n_keys - d.window);
    n_set = ns + max(0, n_keys - wlo);
  } else {
    n_set = n_keys;
  }
  const int per = (n_set + n_splits - 1) / n_splits;
  const int t_lo = split * per;
  const int t_hi = min(n_set, t_lo + per);

  // queries of the group, pre-scaled so that logits are in log2 units
  float qf[G][8];
  {
    const float sc = d.sm_scale * kLog2e;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 v = ld_nc_v4(q + ((int64_t)r * d.n_q + qh0 + g) * kHeadDim + l16 * 8);
      unpack8(v, qf[g]);
#pragma unroll
      for (int i = 0; i < 8; ++i) qf[g][i] *= sc;
    }
  }
  float m_run[G], l_run[G], acc[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_run[g] = -INFINITY;
    l_run[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;
  }
  const int64_t bt_base = (int64_t)seq * cv.max_pages;

  // Where the rows of a batch of tokens live (list entry -> block table -> offset) is resolved one batch ahead, so
  // that these two dependent loads are in flight together with the K / V rows of the current batch.
  int64_t off_n[kUnroll];
  bool ok_n[kUnroll];
  auto resolve = [&](int tb) {
#pragma unroll
    for (int x = 0; x < kUnroll; ++x) {
      const int t = tb + hw + x * kStreams;
      ok_n[x] = t < t_hi;
      off_n[x] = 0;
      if (ok_n[x]) {
        int tok;
        if (SET == kSetList) {
          tok = __ldg(ids + t);
          if (tok < 0 || tok >= n_keys) {
            set_status(status, RTP_ERR_INVALID);
            ok_n[x] = false;
          }
        } else if (SET == kSetLocal) {
          tok = t < ns ? t : wlo + (t - ns);
        } else {
          tok = t;
        }
        if (ok_n[x]) {
          const int phys = safe_phys(cv, bt_base + (tok >> kPageShift), status);
          off_n[x] = (((int64_t)phys * cv.n_kv + kvh) * kPage + (tok & (kPage - 1))) * kHeadDim + l16 * 8;
        }
      }
    }
  };
  // (only lists have the extra dependent load; the other sets resolve in place and keep their register count)
  if (SET == kSetList) resolve(t_lo + warp * 2);
  for (int tb = t_lo + warp * 2; tb < t_hi; tb += kStreams * kUnroll) {
    if (SET != kSetList) resolve(tb);
    uint4 kr[kUnroll], vr[kUnroll];
    bool ok[kUnroll];
#pragma unroll
    for (int x = 0; x < kUnroll; ++x) {
      ok[x] = ok_n[x];
      kr[x] = make_uint4(0, 0, 0, 0);
      vr[x] = make_uint4(0, 0, 0, 0);
      if (ok[x]) {
        kr[x] = ld_stream_v4(cv.k + off_n[x]);
        vr[x] = ld_stream_v4(cv.v + off_n[x]);
      }
    }
    if (SET == kSetList) resolve(tb + kStreams * kUnroll);
    float logit[kUnroll][G];
#pragma unroll
    for (int x = 0; x < kUnroll; ++x) {
      float kf[8];
      unpack8(kr[x], kf);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s = fmaf(qf[g][i], kf[i], s);
        s += __shfl_xor_sync(0xffffffffu, s, 8);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        logit[x][g] = ok[x] ? s : -INFINITY;
      }
    }
    float pw[kUnroll][G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float mx = m_run[g];
#pragma unroll
      for (int x = 0; x < kUnroll; ++x) mx = fmaxf(mx, logit[x][g]);
      if (mx == -INFINITY) {
#pragma unroll
        for (int x = 0; x < kUnroll; ++x) pw[x][g] = 0.f;
        continue;
      }
      const float corr = fast_ex2(m_run[g] - mx);
      float ls = l_run[g] * corr;
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[g][i] *= corr;
#pragma unroll
      for (int x = 0; x < kUnroll; ++x) {
        pw[x][g] = fast_ex2(logit[x][g] - mx);
        ls += pw[x][g];
      }
      l_run[g] = ls;
      m_run[g] = mx;
    }
#pragma unroll
    for (int x = 0; x < kUnroll; ++x) {
      float vf[8];
      unpack8(vr[x], vf);
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] = fmaf(pw[x][g], vf[i], acc[g][i]);
    }
  }

  // merge the eight streams of the CTA
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int i = 0; i < 8; ++i) red[stream][g][l16 * 8 + i] = acc[g][i];
    if (l16 == 0) {
      red[stream][g][kHeadDim] = m_run[g];
      red[stream][g][kHeadDim + 1] = l_run[g];
    }
  }
  __syncthreads();
  const int dim = threadIdx.x;  // 128 threads = 128 dims
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float mt = -INFINITY;
#pragma unroll
    for (int s = 0; s < kStreams; ++s) mt = fmaxf(mt, red[s][g][kHeadDim]);
    float lt = 0.f, a = 0.f;
    if (mt != -INFINITY) {
#pragma unroll
      for (int s = 0; s < kStreams; ++s) {
        const float w = fast_ex2(red[s][g][kHeadDim] - mt);
        lt += red[s][g][kHeadDim + 1] * w;
        a += red[s][g][dim] * w;
      }
    }
    const int64_t oh = (int64_t)r * d.n_q + qh0 + g;
    if (n_splits == 1) {
      out[oh * kHeadDim + dim] = __float2bfloat16_rn(lt > 0.f ? a / lt : 0.f);
      if (lse && dim == 0) lse[oh] = lt > 0.f ? (mt + log2f(lt)) * kLn2 : -INFINITY;
    } else {
      float* p = partial + (((int64_t)blockIdx.x * G + g) * n_splits + split) * kPartial;
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
  const int64_t unit = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t r = unit / n_units;
  const int u = unit % n_units;
  const int qh = (SET == kSetList) ? hm.ret_q_head[u] : hm.kv_list[u] * d.group + g;
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

int plan_splits(int64_t units, int64_t max_set, int sm_count) {
  if (units <= 0) return 1;
  int64_t want = (8LL * sm_count + units - 1) / units;
  int64_t cap = (max_set + 255) / 256;  // at least 256 tokens per CTA
  int64_t s = want < cap ? want : cap;
  if (s < 1) s = 1;
  if (s > 512) s = 512;
  return (int)s;
}

int64_t max_set_len(const Dims& d, int set, int64_t sel_stride, int64_t max_len) {
  if (set == kSetList) return sel_stride < max_len ? sel_stride : max_len;
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
  attn_rows_kernel<G, SET><<<grid, kThreads, 0, st>>>(cv, d, hm, rows, n_units, q, sel_idx, sel_stride, sel_count,
                                                      out, lse, partial, n_splits, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || n_splits == 1) return e;
  attn_merge_kernel<SET><<<(unsigned)(rows.R * n_units * G), kHeadDim, 0, st>>>(d, hm, n_units, G, partial,
                                                                                n_splits, out, lse);
  return cudaGetLastError();
}

}  // namespace

size_t attn_rows_workspace_bytes(const Dims& d, int64_t R, int n_units, int group, int sm_count, int64_t max_len) {
  if (R <= 0 || n_units <= 0) return 0;
  const int n_splits = plan_splits(R * n_units, max_len, sm_count);
  return (size_t)R * n_units * group * n_splits * kPartial * sizeof(float);
}

cudaError_t launch_attn_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows, int set,
                             const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                             const int32_t* sel_count, __nv_bfloat16* out, float* lse, void* ws, size_t ws_bytes,
                             int64_t max_len, int32_t* status, int sm_count, cudaStream_t st) {
  const int n_units = set == kSetList ? d.n_ret : hm.n_kv_list;
  if (rows.R == 0 || n_units == 0) return cudaSuccess;
  const int G = set == kSetList ? 1 : d.group;
  int n_splits = plan_splits(rows.R * n_units, max_set_len(d, set, sel_stride, max_len), sm_count);
  // never plan more splits than the workspace holds
  const size_t per_split = (size_t)rows.R * n_units * G * kPartial * sizeof(float);
  if (n_splits > 1 && (size_t)n_splits * per_split > ws_bytes) n_splits = (int)(ws_bytes / per_split);
  if (n_splits < 1) n_splits = 1;
  float* partial = reinterpret_cast<float*>(ws);
#define RTP_LAUNCH(GG, SS)                                                                                   \
  return launch_typed<GG, SS>(cv, d, hm, rows, n_units, q, sel_idx, sel_stride, sel_count, out, lse, partial, \
                              n_splits, status, st)
  if (set == kSetList) RTP_LAUNCH(1, kSetList);
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
constexpr size_t kStaticScratchBytes = 1u << 20;
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
  const int n_splits = plan_splits(rows.R * d.n_ret, max_set_len(d, kSetList, sel_stride, max_len), sm_count);
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
