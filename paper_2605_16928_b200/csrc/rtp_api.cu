// C ABI: argument validation, head-map construction, workspace planning, kernel launches.
#include <cstdio>
#include <cstring>
#include <string>

#include "rtp_internal.cuh"

struct rtp_ctx {
  int device;
  int sm_count;
  int cc_major, cc_minor;
  unsigned long long wait_ns = 2000000000ull;   // limit of the bounded device-side waits
  int wait_test = 0;                            // rtp_debug_wait_test
  int select_path = 0;                          // rtp_debug_select_path
  std::string last_error;
};

namespace {

using namespace rtp;

rtp_status fail(rtp_ctx* ctx, rtp_status code, const char* msg) {
  if (ctx) ctx->last_error = msg;
  return code;
}

rtp_status cuda_fail(rtp_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
  return RTP_ERR_CUDA;
}

// Any of the selectable variants of the decode selection (fixed budget, forced positions) is on.
bool variant_set(const Dims& d) { return d.top_k > 0 || d.force_sink > 0 || d.force_recent > 0; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates the parameter block and fills the device-side views.  Returns NULL on success, else a message.
const char* check_params(const rtp_params* p, Dims* d, HeadMaps* hm) {
  if (!p) return "params is NULL";
  if (p->head_dim != kHeadDim) return "head_dim must be 128";
  if (p->index_dim != kIndexDim) return "index_dim must be 16";
  if (p->page_size != kPage) return "page_size must be 64";
  if (p->n_kv_heads <= 0 || p->n_q_heads <= 0 || p->n_q_heads > RTP_MAX_Q_HEADS) return "bad head counts";
  if (p->n_q_heads % p->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (p->n_index_heads < 0 || p->n_index_heads > RTP_MAX_INDEX_HEADS) return "bad n_index_heads";
  if (p->n_ret_q_heads < 0 || p->n_ret_q_heads > p->n_q_heads) return "bad n_ret_q_heads";
  if (p->n_local_kv_heads < 0 || p->n_local_kv_heads > p->n_kv_heads) return "bad n_local_kv_heads";
  if (p->n_ret_q_heads > 0 && (!p->ret_q_heads || !p->q_head_to_index_head || !p->index_head_kv))
    return "head map pointer is NULL";
  if (p->n_local_kv_heads > 0 && !p->local_kv_heads) return "local_kv_heads is NULL";
  if (!(p->top_p > 0.0f) || !(p->top_p <= 1.0f)) return "top_p must be in (0, 1]";
  if (!(p->score_scale > 0.0f) || !(p->score_scale < 1e30f)) return "score_scale must be positive and finite";
  if (!(p->sm_scale > 0.0f) || !(p->sm_scale < 1e30f)) return "sm_scale must be positive and finite";
  if (p->n_sink < 0 || p->window < 1) return "n_sink must be >= 0 and window >= 1";
  if (p->top_k < 0) return "top_k must be >= 0";
  if (p->force_sink < 0 || p->force_recent < 0 || (int64_t)p->force_sink + p->force_recent > 65536)
    return "force_sink and force_recent must be >= 0 and sum to at most 65536";
  d->n_q = p->n_q_heads;
  d->n_kv = p->n_kv_heads;
  d->n_ih = p->n_index_heads;
  d->n_ret = p->n_ret_q_heads;
  d->group = p->n_q_heads / p->n_kv_heads;
  d->n_sink = p->n_sink;
  d->window = p->window;
  d->top_p = p->top_p;
  d->top_k = p->top_k;
  d->force_sink = p->force_sink;
  d->force_recent = p->force_recent;
  d->score_scale = p->score_scale;
  d->sm_scale = p->sm_scale;
  d->wait_ns = 2000000000ull;
  d->wait_test = 0;
  d->select_path = 0;
  std::memset(hm, 0, sizeof(*hm));
  for (int j = 0; j < p->n_index_heads; ++j) {
    const int kv = p->index_head_kv[j];
    if (kv < 0 || kv >= p->n_kv_heads) return "index_head_kv out of range";
    hm->ih_kv[j] = (uint8_t)kv;
  }
  for (int i = 0; i < p->n_ret_q_heads; ++i) {
    const int h = p->ret_q_heads[i], j = p->q_head_to_index_head[i];
    if (h < 0 || h >= p->n_q_heads) return "ret_q_heads out of range";
    if (j < 0 || j >= p->n_index_heads) return "q_head_to_index_head out of range";
    if (hm->ih_nheads[j] >= RTP_MAX_HEADS_PER_INDEX_HEAD) return "too many query heads on one index head";
    hm->ret_q_head[i] = (uint8_t)h;
    hm->q2ih[i] = (uint8_t)j;
    hm->slot_in_ih[i] = hm->ih_nheads[j];
    hm->ih_heads[j][hm->ih_nheads[j]++] = (uint8_t)i;
  }
  for (int i = 0; i < p->n_local_kv_heads; ++i) {
    const int kv = p->local_kv_heads[i];
    if (kv < 0 || kv >= p->n_kv_heads) return "local_kv_heads out of range";
  }
  return nullptr;
}

const char* check_cache(const rtp_cache* c, const rtp_params* p, bool need_kv, bool need_ikey, CacheView* cv) {
  if (!c) return "cache is NULL";
  if (c->num_pages <= 0 || c->batch <= 0 || c->max_pages <= 0) return "cache sizes must be positive";
  if (!c->block_table || !c->seq_lens) return "block_table / seq_lens is NULL";
  if (need_kv && (!c->k_pages || !c->v_pages)) return "k_pages / v_pages is NULL";
  if (need_ikey && !c->ikey_pages) return "ikey_pages is NULL";
  if (!aligned16(c->k_pages) || !aligned16(c->v_pages) || !aligned16(c->ikey_pages)) return "cache pages must be 16-byte aligned";
  if (p->n_kv_heads > 32) return "more than 32 KV heads";
  cv->k = reinterpret_cast<const __nv_bfloat16*>(c->k_pages);
  cv->v = reinterpret_cast<const __nv_bfloat16*>(c->v_pages);
  cv->ikey = reinterpret_cast<__nv_bfloat16*>(c->ikey_pages);
  cv->block_table = c->block_table;
  cv->seq_lens = c->seq_lens;
  cv->num_pages = c->num_pages;
  cv->batch = c->batch;
  cv->max_pages = c->max_pages;
  cv->n_kv = p->n_kv_heads;
  cv->n_ih = p->n_index_heads;
  cv->cap_tokens = (int32_t)std::min<int64_t>((int64_t)c->max_pages * kPage, 0x7fffffff);
  cv->sink_pages = 0;
  cv->ring_pages = 0;
  if (c->ikey_format != RTP_IKEY_BF16 && c->ikey_format != RTP_IKEY_E4M3) return "unknown ikey_format";
  cv->ikey_fp8 = c->ikey_format == RTP_IKEY_E4M3;
  for (int h = 0; h < 32; ++h) cv->kv_slot[h] = h < p->n_kv_heads ? (uint8_t)h : (uint8_t)0xff;
  if (c->k_local_pages) {
    // truncated layout: the main pool holds the KV heads that are not local, in increasing order
    if (!c->v_local_pages || !c->local_block_table) return "v_local_pages / local_block_table is NULL";
    if (!aligned16(c->k_local_pages) || !aligned16(c->v_local_pages)) return "local cache pages must be 16-byte aligned";
    if (c->n_local_pages <= 0 || c->ring_pages <= 0 || c->sink_pages < 0) return "local cache sizes must be positive";
    if ((int64_t)c->sink_pages * kPage < p->n_sink) return "sink_pages does not cover n_sink";
    if (p->n_local_kv_heads <= 0) return "a local cache without local KV heads";
    bool local[32] = {};
    for (int i = 0; i < p->n_local_kv_heads; ++i) local[p->local_kv_heads[i]] = true;
    // a mixed group (retrieval and local query heads on one KV head) needs that head's whole history
    const int group = p->n_q_heads / p->n_kv_heads;
    for (int i = 0; i < p->n_ret_q_heads; ++i)
      if (local[p->ret_q_heads[i] / group]) return "a KV head with retrieval query heads cannot live in the truncated pool";
    int n_main = 0;
    for (int h = 0; h < p->n_kv_heads; ++h) cv->kv_slot[h] = local[h] ? (uint8_t)0xff : (uint8_t)n_main++;
    cv->n_kv = n_main;
  }
  return nullptr;
}

// The local heads' pool of a truncated cache as a view of its own (the index-key cache is not reachable through it).
CacheView local_view(const CacheView& main, const rtp_cache* c, const rtp_params* p) {
  CacheView v = main;
  v.k = reinterpret_cast<const __nv_bfloat16*>(c->k_local_pages);
  v.v = reinterpret_cast<const __nv_bfloat16*>(c->v_local_pages);
  v.ikey = nullptr;
  v.block_table = c->local_block_table;
  v.num_pages = c->n_local_pages;
  v.max_pages = c->sink_pages + c->ring_pages;
  v.n_kv = p->n_local_kv_heads;
  v.sink_pages = c->sink_pages;
  v.ring_pages = c->ring_pages;
  for (int h = 0; h < 32; ++h) v.kv_slot[h] = 0xff;
  for (int i = 0; i < p->n_local_kv_heads; ++i) v.kv_slot[p->local_kv_heads[i]] = (uint8_t)i;
  return v;
}

const char* check_rows(const int32_t* row_seq, const int32_t* row_pos, int32_t seq_id, int32_t q_start, int64_t R,
                       const rtp_cache* c, Rows* rows, int64_t* max_len) {
  if (R < 0) return "row count is negative";
  if ((row_seq == nullptr) != (row_pos == nullptr)) return "row_seq and row_pos must both be given or both be NULL";
  rows->seq = row_seq;
  rows->pos = row_pos;
  rows->seq_id = seq_id;
  rows->q_start = q_start;
  rows->R = R;
  const int64_t cap = (int64_t)c->max_pages * kPage;
  if (!row_seq) {
    if (seq_id < 0 || seq_id >= c->batch) return "seq_id out of range";
    if (q_start < 0 || q_start + R > cap) return "chunk exceeds the block table";
    *max_len = q_start + R;
  } else {
    *max_len = cap;
  }
  return nullptr;
}

struct WsCarver {
  char* base;
  size_t off = 0;
  explicit WsCarver(void* p) : base(reinterpret_cast<char*>(p)) {}
  void* take(size_t n) {
    void* r = base ? base + off : nullptr;
    off += (n + 255) & ~(size_t)255;
    return r;
  }
};

size_t qt_bytes(const Dims& d, int64_t R) { return (size_t)R * d.n_ret * kIndexDim * sizeof(__nv_bfloat16); }

// SM count assumed when sizes are asked for without a device to query (a B200 has 148).
constexpr int kFallbackSm = 148;

}  // namespace

extern "C" {

int32_t rtp_version(void) { return 100; }

size_t rtp_struct_bytes(int32_t what) { return what == 0 ? sizeof(rtp_params) : (what == 1 ? sizeof(rtp_cache) : 0); }

rtp_status rtp_create(rtp_ctx** out_ctx) {
  if (!out_ctx) return RTP_ERR_INVALID;
  *out_ctx = nullptr;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return RTP_ERR_CUDA;
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess) return RTP_ERR_CUDA;
  if (prop.major != 10) return RTP_ERR_UNSUPPORTED;
  rtp_ctx* c = new rtp_ctx();
  c->device = dev;
  c->sm_count = prop.multiProcessorCount;
  c->cc_major = prop.major;
  c->cc_minor = prop.minor;
  *out_ctx = c;
  return RTP_OK;
}

void rtp_destroy(rtp_ctx* ctx) { delete ctx; }

rtp_status rtp_debug_select_path(rtp_ctx* ctx, int32_t path) {
  if (!ctx || path < 0 || path > 1) return RTP_ERR_INVALID;
  ctx->select_path = path;
  return RTP_OK;
}

const char* rtp_last_error(const rtp_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "no context"; }

rtp_status rtp_debug_wait_test(rtp_ctx* ctx, int64_t wait_limit_ns, int32_t drop_first_key_signal) {
  if (!ctx || wait_limit_ns <= 0) return RTP_ERR_INVALID;
  ctx->wait_ns = (unsigned long long)wait_limit_ns;
  ctx->wait_test = drop_first_key_signal ? 1 : 0;
  return RTP_OK;
}

size_t rtp_workspace_bytes(const rtp_params* params, int64_t rows, int64_t max_seq_len) {
  Dims d;
  HeadMaps hm;
  if (check_params(params, &d, &hm) || rows <= 0 || max_seq_len <= 0) return 0;
  WsCarver w(nullptr);
  w.take(qt_bytes(d, rows));
  size_t a = select_rows_workspace_bytes(d, rows, max_seq_len);
  const size_t b = select_chunk_workspace_bytes(d, hm, rows);
  // explicit-row selection keeps 48 KB and one fp32 score per key for every (row, head); beyond 4096 rows only the
  // chunk path is sized
  if (rows > 4096) a = 0;
  size_t m = a > b ? a : b;
  const size_t s = score_workspace_bytes(d, rows, max_seq_len, current_sm_count(kFallbackSm) * 2);
  m = m > s ? m : s;
  const size_t t1 = attn_rows_workspace_bytes(d, rows, d.n_ret, 1, 1024, max_seq_len);
  const size_t t2 = attn_rows_workspace_bytes(d, rows, d.n_kv, d.group, 1024, max_seq_len);
  if (rows <= 4096) {
    const size_t t3 = t2 + ((block_union_bytes(d, rows, max_seq_len) + 255) & ~(size_t)255);   // block-wise decode
    m = m > t1 ? m : t1;
    m = m > t3 ? m : t3;
  }
  w.take(m);
  return w.off;
}

rtp_status rtp_check_status(rtp_ctx* ctx, const int32_t* status, void* stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
  if (!status) return RTP_OK;
  int32_t h = 0;
  e = cudaMemcpy(&h, status, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMemcpy(status)");
  if (h < 0 || h > RTP_ERR_TIMEOUT) return RTP_ERR_INVALID;
  return (rtp_status)h;
}

#define RTP_COMMON_PROLOGUE(need_kv, need_ikey)                                   \
  if (!ctx) return RTP_ERR_INVALID;                                               \
  Dims d;                                                                         \
  HeadMaps hm;                                                                    \
  CacheView cv;                                                                   \
  if (const char* m_ = check_params(params, &d, &hm)) return fail(ctx, RTP_ERR_INVALID, m_); \
  d.wait_ns = ctx->wait_ns;                                                       \
  d.wait_test = ctx->wait_test;                                                   \
  d.select_path = ctx->select_path;                                               \
  if (const char* m_ = check_cache(cache, params, need_kv, need_ikey, &cv)) return fail(ctx, RTP_ERR_INVALID, m_); \
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

rtp_status rtp_index_keys(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* k_pre,
                          const void* w_k, const int32_t* tok_seq, const int32_t* tok_pos, int64_t T, void* stream) {
  RTP_COMMON_PROLOGUE(false, true)
  if (T < 0) return fail(ctx, RTP_ERR_INVALID, "T is negative");
  if (T == 0) return RTP_OK;
  if (d.n_ih == 0) return fail(ctx, RTP_ERR_INVALID, "no index heads");
  if (!k_pre || !w_k || !tok_seq || !tok_pos) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(k_pre) || !aligned16(w_k)) return fail(ctx, RTP_ERR_INVALID, "k_pre / w_k must be 16-byte aligned");
  cudaError_t e = launch_index_keys(cv, d, reinterpret_cast<const __nv_bfloat16*>(k_pre),
                                    reinterpret_cast<const __nv_bfloat16*>(w_k), tok_seq, tok_pos, T, st);
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_index_keys");
}

rtp_status rtp_kv_append(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* k_new,
                         const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int64_t T,
                         int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  if (T < 0) return fail(ctx, RTP_ERR_INVALID, "T is negative");
  if (T == 0) return RTP_OK;
  if (!k_new || !v_new || !tok_seq || !tok_pos) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(k_new) || !aligned16(v_new)) return fail(ctx, RTP_ERR_INVALID, "k_new / v_new must be 16-byte aligned");
  (void)hm;
  cudaError_t e = cudaSuccess;
  if (cv.n_kv > 0)
    e = launch_kv_append(cv, d.n_kv, reinterpret_cast<const __nv_bfloat16*>(k_new),
                         reinterpret_cast<const __nv_bfloat16*>(v_new), tok_seq, tok_pos, T, status, st);
  if (e == cudaSuccess && cache->k_local_pages)
    e = launch_kv_append(local_view(cv, cache, params), d.n_kv, reinterpret_cast<const __nv_bfloat16*>(k_new),
                         reinterpret_cast<const __nv_bfloat16*>(v_new), tok_seq, tok_pos, T, status, st);
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_kv_append");
}

rtp_status rtp_index_queries(rtp_ctx* ctx, const rtp_params* params, const void* q_pre, const void* w_q, int64_t R,
                             void* qt_out, void* stream) {
  if (!ctx) return RTP_ERR_INVALID;
  Dims d;
  HeadMaps hm;
  if (const char* m = check_params(params, &d, &hm)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R < 0) return fail(ctx, RTP_ERR_INVALID, "R is negative");
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q_pre || !w_q || !qt_out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q_pre) || !aligned16(w_q) || !aligned16(qt_out)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), R,
                                       reinterpret_cast<__nv_bfloat16*>(qt_out), reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_index_queries");
}

rtp_status rtp_index_score(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                           const void* w_q, const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                           float* scores_out, int64_t score_stride, float* row_max_out, float* row_sum_out,
                           void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(false, true)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q_pre || !w_q || !workspace) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q_pre) || !aligned16(w_q) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (scores_out && score_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "score_stride must be positive");
  if (scores_out && score_stride < max_len) max_len = score_stride;
  WsCarver w(workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(w.take(qt_bytes(d, R)));
  void* part = w.take(score_workspace_bytes(d, R, max_len, ctx->sm_count));
  if (w.off > workspace_bytes) return fail(ctx, RTP_ERR_CAPACITY, "workspace too small");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), R, qt, st);
  if (e == cudaSuccess)
    e = launch_index_score(cv, d, hm, rows, qt, max_len, scores_out, score_stride, row_max_out, row_sum_out, part,
                           status, ctx->sm_count, st);
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_index_score");
}

rtp_status rtp_topp_select(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                           const void* w_q, const int32_t* row_seq, const int32_t* row_pos, int32_t seq_id,
                           int32_t q_start, int64_t R, int32_t* sel_idx, int64_t sel_stride, int32_t* sel_count,
                           float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status,
                           void* workspace, size_t workspace_bytes, void* stream) {
  RTP_COMMON_PROLOGUE(false, true)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(row_seq, row_pos, seq_id, q_start, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q_pre || !w_q || !workspace || !sel_count) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q_pre) || !aligned16(w_q) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (sel_idx && sel_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "sel_stride must be positive");
  WsCarver w(workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(w.take(qt_bytes(d, R)));
  const bool chunk = row_seq == nullptr;
  if (chunk && variant_set(d)) return fail(ctx, RTP_ERR_UNSUPPORTED, "top_k / forced positions: row lists only");
  if (chunk && cv.ikey_fp8) return fail(ctx, RTP_ERR_UNSUPPORTED, "8-bit index keys: row form only");
  const size_t sel_off = w.off;
  void* sel_ws = w.take(chunk ? select_chunk_workspace_bytes(d, hm, R) : select_rows_workspace_bytes(d, R, max_len));
  if (w.off > workspace_bytes) return fail(ctx, RTP_ERR_CAPACITY, "workspace too small");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), R, qt, st);
  if (e == cudaSuccess) {
    if (chunk)
      e = launch_select_chunk(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh,
                              sel_tie_last, status, sel_ws, workspace_bytes - sel_off, ctx->sm_count, st);
    else
      e = launch_select_rows(cv, d, hm, rows, qt, max_len, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh,
                             sel_tie_last, status, sel_ws, ctx->sm_count, st);
  }
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_topp_select");
}

rtp_status rtp_sparse_attn_decode(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                  const int32_t* row_seq, const int32_t* row_pos, int64_t R, const int32_t* sel_idx,
                                  int64_t sel_stride, const int32_t* sel_count, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q || !sel_idx || !sel_count || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (sel_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "sel_stride must be positive");
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  cudaError_t e = launch_attn_rows(cv, d, hm, rows, kSetList, reinterpret_cast<const __nv_bfloat16*>(q), sel_idx,
                                   sel_stride, sel_count, reinterpret_cast<__nv_bfloat16*>(out), lse, workspace,
                                   workspace ? workspace_bytes : 0, max_len, status, ctx->sm_count, st);
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_decode");
}

rtp_status rtp_sparse_attn_decode_static(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                         const void* q, const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                                         const int32_t* sel_idx, int64_t sel_stride, const int32_t* sel_count,
                                         void* out, float* lse, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q || !sel_idx || !sel_count || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (sel_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "sel_stride must be positive");
  if (!aligned16(q) || !aligned16(out)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  size_t need = 0;
  cudaError_t e = launch_attn_rows_static(cv, d, hm, rows, reinterpret_cast<const __nv_bfloat16*>(q), sel_idx,
                                          sel_stride, sel_count, reinterpret_cast<__nv_bfloat16*>(out), lse, max_len,
                                          status, ctx->sm_count, &need, st);
  if (e == cudaErrorMemoryAllocation && need > attn_rows_static_scratch_bytes()) {
    char msg[192];
    std::snprintf(msg, sizeof(msg),
                  "rtp_sparse_attn_decode_static: this call needs %zu bytes of split scratch but the built-in "
                  "array holds %zu; use rtp_sparse_attn_decode with a caller workspace or fewer rows",
                  need, attn_rows_static_scratch_bytes());
    return fail(ctx, RTP_ERR_CAPACITY, msg);
  }
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_decode_static");
}

rtp_status rtp_sparse_attn_prefill(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                   const void* q_pre, const void* w_q, int32_t seq_id, int32_t q_start, int64_t C,
                                   const int32_t* sel_idx, int64_t sel_stride, const int32_t* sel_count,
                                   const float* sel_thresh, const int32_t* sel_tie_last, void* out, float* lse,
                                   void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, sel_idx == nullptr)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(nullptr, nullptr, seq_id, q_start, C, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (C == 0 || d.n_ret == 0) return RTP_OK;
  if (!q || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (sel_idx) {
    if (!sel_count || sel_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "sel_count / sel_stride invalid");
    cudaError_t e = launch_attn_rows(cv, d, hm, rows, kSetList, reinterpret_cast<const __nv_bfloat16*>(q), sel_idx,
                                     sel_stride, sel_count, reinterpret_cast<__nv_bfloat16*>(out), lse, workspace,
                                     workspace ? workspace_bytes : 0, max_len, status, ctx->sm_count, st);
    return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_prefill(lists)");
  }
  if (!sel_thresh || !sel_tie_last || !q_pre || !w_q || !workspace)
    return fail(ctx, RTP_ERR_INVALID, "threshold mode needs sel_thresh, sel_tie_last, q_pre, w_q and a workspace");
  if (cv.ikey_fp8) return fail(ctx, RTP_ERR_UNSUPPORTED, "8-bit index keys: list form only");
  if (variant_set(d)) return fail(ctx, RTP_ERR_UNSUPPORTED, "top_k / forced positions: row lists only");
  if (!aligned16(q_pre) || !aligned16(w_q)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  WsCarver w(workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(w.take(qt_bytes(d, C)));
  if (w.off > workspace_bytes) return fail(ctx, RTP_ERR_CAPACITY, "workspace too small");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), C, qt, st);
  if (e == cudaSuccess)
    e = launch_attn_prefill(cv, d, hm, kPrefillSparse, reinterpret_cast<const __nv_bfloat16*>(q), qt, seq_id, q_start,
                            C, sel_thresh, sel_tie_last, reinterpret_cast<__nv_bfloat16*>(out), lse, status,
                            ctx->sm_count, st);
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_prefill");
}

size_t rtp_block_workspace_bytes(const rtp_params* params, int64_t rows, int64_t max_seq_len) {
  Dims d;
  HeadMaps hm;
  if (check_params(params, &d, &hm) || rows <= 0 || max_seq_len <= 0) return 0;
  WsCarver w(nullptr);
  w.take(qt_bytes(d, rows));
  w.take(select_blocks_workspace_bytes(d, hm, rows, max_seq_len, current_sm_count(kFallbackSm)));
  w.take(select_rows_blocks_workspace_bytes(d, rows, max_seq_len));   // (the row form; one buffer serves either)
  return w.off;
}

rtp_status rtp_topp_select_blocks_rows(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                                       const void* w_q, const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                                       int32_t* block_idx, int64_t block_stride, int32_t* sel_count, float* sel_mass,
                                       float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* workspace,
                                       size_t workspace_bytes, void* stream) {
  RTP_COMMON_PROLOGUE(false, true)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q_pre || !w_q || !workspace || !sel_count) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q_pre) || !aligned16(w_q) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (block_idx && block_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "block_stride must be positive");
  if (variant_set(d)) return fail(ctx, RTP_ERR_UNSUPPORTED, "top_k / forced positions: token lists only");
  WsCarver w(workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(w.take(qt_bytes(d, R)));
  void* sel_ws = w.take(select_rows_blocks_workspace_bytes(d, R, max_len));
  if (w.off > workspace_bytes) return fail(ctx, RTP_ERR_CAPACITY, "workspace too small");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), R, qt, st);
  if (e == cudaSuccess)
    e = launch_select_rows_blocks(cv, d, hm, rows, qt, max_len, block_idx, block_stride, sel_count, sel_mass, sel_thresh,
                                  sel_tie_last, status, sel_ws, ctx->sm_count, st);
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "more than 16384 blocks per row");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_topp_select_blocks_rows");
}

rtp_status rtp_sparse_attn_decode_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                         const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                                         const int32_t* block_idx, int64_t block_stride, const int32_t* block_count,
                                         void* out, float* lse, void* workspace, size_t workspace_bytes,
                                         int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || d.n_ret == 0) return RTP_OK;
  if (!q || !block_idx || !block_count || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (block_stride <= 0) return fail(ctx, RTP_ERR_INVALID, "block_stride must be positive");
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  // With a workspace the pages of a KV head's query heads are merged into one flagged list per (row, KV head) and the
  // whole group is attended in one pass over that union (Section 3.2: the memory a KV head needs is the union of its
  // heads' sets): shared pages are read once.  Without one every head gathers its own pages.
  cudaError_t e;
  const size_t uni_bytes = block_union_bytes(d, R, max_len);
  const bool grouped = workspace && workspace_bytes > uni_bytes && (d.group == 1 || d.group == 2 || d.group == 4 || d.group == 8);
  if (grouped) {
    bool is_ret[RTP_MAX_Q_HEADS] = {};
    bool kv_used[32] = {};
    for (int i = 0; i < d.n_ret; ++i) {
      is_ret[hm.ret_q_head[i]] = true;
      kv_used[hm.ret_q_head[i] / d.group] = true;
    }
    hm.n_kv_list = 0;
    for (int kv = 0; kv < d.n_kv; ++kv)
      if (kv_used[kv]) hm.kv_list[hm.n_kv_list++] = (uint8_t)kv;
    for (int h = 0; h < d.n_q; ++h)   // the group's heads that are not retrieval heads are computed but not written
      if (!is_ret[h]) hm.skip_q[h >> 5] |= 1u << (h & 31);
    int32_t *uni_idx = nullptr, *uni_cnt = nullptr;
    int64_t uni_stride = 0;
    e = launch_block_union(cv, d, hm, rows, block_idx, block_stride, block_count, max_len, workspace, &uni_idx, &uni_stride,
                           &uni_cnt, status, st);
    if (e == cudaSuccess)
      e = launch_attn_rows(cv, d, hm, rows, kSetUnion, reinterpret_cast<const __nv_bfloat16*>(q), uni_idx, uni_stride, uni_cnt,
                           reinterpret_cast<__nv_bfloat16*>(out), lse, reinterpret_cast<char*>(workspace) + uni_bytes,
                           workspace_bytes - uni_bytes, max_len, status, ctx->sm_count, st);
  } else {
    e = launch_attn_rows(cv, d, hm, rows, kSetPages, reinterpret_cast<const __nv_bfloat16*>(q), block_idx, block_stride,
                         block_count, reinterpret_cast<__nv_bfloat16*>(out), lse, workspace,
                         workspace ? workspace_bytes : 0, max_len, status, ctx->sm_count, st);
  }
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_decode_blocks");
}

rtp_status rtp_topp_select_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                                  const void* w_q, int32_t seq_id, int32_t q_start, int64_t C, uint32_t* block_mask,
                                  int64_t mask_words, int32_t* sel_count, float* sel_mass, float* sel_thresh,
                                  int32_t* sel_tie_last, int32_t* status, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  RTP_COMMON_PROLOGUE(false, true)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(nullptr, nullptr, seq_id, q_start, C, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (C == 0 || d.n_ret == 0) return RTP_OK;
  if (!q_pre || !w_q || !workspace || !sel_count || !block_mask) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q_pre) || !aligned16(w_q) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (mask_words * 32 < ((int64_t)q_start + C + kPage - 1) / kPage) return fail(ctx, RTP_ERR_CAPACITY, "mask_words too small for the chunk's pages");
  if (cv.ikey_fp8) return fail(ctx, RTP_ERR_UNSUPPORTED, "8-bit index keys: row form of the selection only");
  if (variant_set(d)) return fail(ctx, RTP_ERR_UNSUPPORTED, "top_k / forced positions: row lists only");
  WsCarver w(workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(w.take(qt_bytes(d, C)));
  const size_t sel_off = w.off;
  void* sel_ws = w.take(select_blocks_workspace_bytes(d, hm, C, (int64_t)q_start + C, ctx->sm_count));
  if (w.off > workspace_bytes) return fail(ctx, RTP_ERR_CAPACITY, "workspace too small");
  cudaError_t e = launch_index_queries(d, hm, reinterpret_cast<const __nv_bfloat16*>(q_pre),
                                       reinterpret_cast<const __nv_bfloat16*>(w_q), C, qt, st);
  if (e == cudaSuccess)
    e = launch_select_blocks(cv, d, hm, rows, qt, block_mask, mask_words, sel_count, sel_mass, sel_thresh, sel_tie_last,
                             status, sel_ws, workspace_bytes - sel_off, ctx->sm_count, st);
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_topp_select_blocks");
}

rtp_status rtp_sparse_attn_prefill_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                          int32_t seq_id, int32_t q_start, int64_t C, const uint32_t* block_mask,
                                          int64_t mask_words, void* out, float* lse, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(nullptr, nullptr, seq_id, q_start, C, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (C == 0 || d.n_ret == 0) return RTP_OK;
  if (!q || !out || !block_mask) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q) || !aligned16(out)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (mask_words * 32 < ((int64_t)q_start + C + kPage - 1) / kPage) return fail(ctx, RTP_ERR_INVALID, "mask_words too small for the chunk's pages");
  cudaError_t e = launch_attn_prefill(cv, d, hm, kPrefillBlocks, reinterpret_cast<const __nv_bfloat16*>(q), nullptr, seq_id,
                                      q_start, C, nullptr, nullptr, reinterpret_cast<__nv_bfloat16*>(out), lse, status,
                                      ctx->sm_count, st, block_mask, mask_words);
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_sparse_attn_prefill_blocks");
}

rtp_status rtp_local_attn(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                          const int32_t* row_seq, const int32_t* row_pos, int32_t seq_id, int32_t q_start, int64_t R,
                          void* out, float* lse, void* workspace, size_t workspace_bytes, int32_t* status,
                          void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(row_seq, row_pos, seq_id, q_start, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (R == 0 || params->n_local_kv_heads == 0) return RTP_OK;
  if (!q || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  hm.n_kv_list = params->n_local_kv_heads;
  for (int i = 0; i < hm.n_kv_list; ++i) hm.kv_list[i] = (uint8_t)params->local_kv_heads[i];
  // a mixed group: its retrieval heads are written by the sparse call, not by this one
  for (int i = 0; i < d.n_ret; ++i) hm.skip_q[hm.ret_q_head[i] >> 5] |= 1u << (hm.ret_q_head[i] & 31);
  if (cache->k_local_pages) {
    // truncated cache: the local heads' ring must still hold the window of the call's oldest row
    const int64_t ahead = row_seq ? 0 : R;   // a chunk is appended before it is attended
    if ((int64_t)cache->ring_pages * kPage < (int64_t)d.window + ahead + kPage)
      return fail(ctx, RTP_ERR_CAPACITY, "ring_pages too small for the window (plus the chunk) of this call");
    cv = local_view(cv, cache, params);
  }
  cudaError_t e;
  if (row_seq) {
    if (d.group != 1 && d.group != 2 && d.group != 4 && d.group != 8)
      return fail(ctx, RTP_ERR_UNSUPPORTED, "GQA group size must be 1, 2, 4 or 8");
    e = launch_attn_rows(cv, d, hm, rows, kSetLocal, reinterpret_cast<const __nv_bfloat16*>(q), nullptr, 0, nullptr,
                         reinterpret_cast<__nv_bfloat16*>(out), lse, workspace, workspace ? workspace_bytes : 0,
                         max_len, status, ctx->sm_count, st);
  } else {
    e = launch_attn_prefill(cv, d, hm, kPrefillLocal, reinterpret_cast<const __nv_bfloat16*>(q), nullptr, seq_id,
                            q_start, R, nullptr, nullptr, reinterpret_cast<__nv_bfloat16*>(out), lse, status,
                            ctx->sm_count, st);
  }
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_local_attn");
}

static const char* fill_kv_list(const rtp_params* params, const int32_t* kv_heads, int32_t n_heads, HeadMaps* hm) {
  if (!kv_heads) {
    hm->n_kv_list = params->n_kv_heads;
    for (int i = 0; i < hm->n_kv_list; ++i) hm->kv_list[i] = (uint8_t)i;
    return nullptr;
  }
  if (n_heads < 0 || n_heads > params->n_kv_heads) return "bad n_heads";
  hm->n_kv_list = n_heads;
  for (int i = 0; i < n_heads; ++i) {
    if (kv_heads[i] < 0 || kv_heads[i] >= params->n_kv_heads) return "kv_heads out of range";
    hm->kv_list[i] = (uint8_t)kv_heads[i];
  }
  return nullptr;
}

rtp_status rtp_dense_attn_prefill(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                  int32_t seq_id, int32_t q_start, int64_t C, const int32_t* kv_heads,
                                  int32_t n_heads, void* out, float* lse, int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (const char* m = check_rows(nullptr, nullptr, seq_id, q_start, C, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (const char* m = fill_kv_list(params, kv_heads, n_heads, &hm)) return fail(ctx, RTP_ERR_INVALID, m);
  for (int i = 0; i < hm.n_kv_list; ++i)
    if (cv.kv_slot[hm.kv_list[i]] == 0xff)
      return fail(ctx, RTP_ERR_UNSUPPORTED, "the cache is truncated for local heads: a dense call may only name the other KV heads");
  if (C == 0 || hm.n_kv_list == 0) return RTP_OK;
  if (!q || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q) || !aligned16(out)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  cudaError_t e = launch_attn_prefill(cv, d, hm, kPrefillDense, reinterpret_cast<const __nv_bfloat16*>(q), nullptr,
                                      seq_id, q_start, C, nullptr, nullptr, reinterpret_cast<__nv_bfloat16*>(out),
                                      lse, status, ctx->sm_count, st);
  if (e == cudaErrorNotSupported) return fail(ctx, RTP_ERR_UNSUPPORTED, "not implemented in this build");
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_dense_attn_prefill");
}

rtp_status rtp_dense_attn_decode(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                 const int32_t* row_seq, const int32_t* row_pos, int64_t R, const int32_t* kv_heads,
                                 int32_t n_heads, void* out, float* lse, void* workspace, size_t workspace_bytes,
                                 int32_t* status, void* stream) {
  RTP_COMMON_PROLOGUE(true, false)
  Rows rows;
  int64_t max_len = 0;
  if (!row_seq || !row_pos) return fail(ctx, RTP_ERR_INVALID, "row_seq / row_pos is NULL");
  if (const char* m = check_rows(row_seq, row_pos, 0, 0, R, cache, &rows, &max_len)) return fail(ctx, RTP_ERR_INVALID, m);
  if (const char* m = fill_kv_list(params, kv_heads, n_heads, &hm)) return fail(ctx, RTP_ERR_INVALID, m);
  for (int i = 0; i < hm.n_kv_list; ++i)
    if (cv.kv_slot[hm.kv_list[i]] == 0xff)
      return fail(ctx, RTP_ERR_UNSUPPORTED, "the cache is truncated for local heads: a dense call may only name the other KV heads");
  if (R == 0 || hm.n_kv_list == 0) return RTP_OK;
  if (!q || !out) return fail(ctx, RTP_ERR_INVALID, "NULL argument");
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return fail(ctx, RTP_ERR_INVALID, "misaligned pointer");
  if (d.group != 1 && d.group != 2 && d.group != 4 && d.group != 8)
    return fail(ctx, RTP_ERR_UNSUPPORTED, "GQA group size must be 1, 2, 4 or 8");
  cudaError_t e = launch_attn_rows(cv, d, hm, rows, kSetDense, reinterpret_cast<const __nv_bfloat16*>(q), nullptr, 0,
                                   nullptr, reinterpret_cast<__nv_bfloat16*>(out), lse, workspace,
                                   workspace ? workspace_bytes : 0, max_len, status, ctx->sm_count, st);
  return e == cudaSuccess ? RTP_OK : cuda_fail(ctx, e, "rtp_dense_attn_decode");
}

}  // extern "C"
