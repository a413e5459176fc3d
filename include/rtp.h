/*
 * rtp.h - C ABI of the sparse-attention hot path (sm_100a).
 *
 * The library implements the inference-time attention mechanism of the paper's
 * Section 3.2: a 16-dimensional token indexer (Eq. 4), a query-dependent top-p
 * selection on the softmax mass of the indexer scores (Eq. 5, "Top-P"), exact
 * attention restricted to the selected tokens on retrieval heads (Eq. 5), and
 * attention-sink + sliding-window attention on local heads (Section 3.2,
 * Table 2), plus dense causal attention as the in-library comparator.
 *
 * General contract
 * ----------------
 * - Every pointer marked DEVICE points to global memory of the current CUDA
 *   device and must be 16-byte aligned; every pointer marked HOST is ordinary
 *   host memory read during the call.  All tensors are dense, row-major.
 * - The library allocates no device memory.  Caches, outputs, selection
 *   buffers and scratch ("workspace", size from rtp_workspace_bytes) belong to
 *   the caller.  Workspace contents are undefined after a call; two calls that
 *   may overlap on the GPU must not share a workspace.
 * - Calls are asynchronous on the CUDA stream passed as `stream` (a
 *   cudaStream_t cast to void*, NULL = default stream).
 * - Every call returns an rtp_status.  Errors detectable on the host (NULL or
 *   misaligned pointers, unsupported sizes, p outside (0,1]) are returned before
 *   anything is launched.  Conditions only visible on the device (a selection
 *   list that overflows, a row position beyond its sequence) are reported by
 *   writing the largest rtp_status code seen into the caller's DEVICE int32
 *   `status` word (which the caller zeroes); kernels never trap.
 * - bf16 = 16-bit brain float bit patterns.  Fixed sizes: head_dim 128,
 *   index_dim 16, page_size 64.
 *
 * Head conventions: query head h reads KV head h / (n_q_heads / n_kv_heads).
 * The partition into retrieval and local heads is over QUERY heads (Section 3.2): a KV head may be listed in
 * local_kv_heads while some query heads of its group are retrieval heads (a mixed group).  rtp_local_attn then
 * writes only the group's query heads that are not retrieval heads, the decode calls and the list form of
 * rtp_sparse_attn_prefill serve its retrieval heads; the threshold and block-wise forms of the prefill attention
 * need index heads that cover whole groups (RTP_ERR_UNSUPPORTED otherwise), and such a KV head cannot live in the
 * truncated pool of rtp_cache (RTP_ERR_INVALID).
 * Retrieval query heads are listed in rtp_params.ret_q_heads; entry i has its
 * own W_q[i] and its own selection, and scores against the index-key stream
 * q_head_to_index_head[i].  Index head j projects the pre-RoPE keys of KV head
 * index_head_kv[j] with W_k[j].
 */
#ifndef RTP_H_
#define RTP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RTP_HEAD_DIM 128
#define RTP_INDEX_DIM 16
#define RTP_PAGE_SIZE 64
#define RTP_MAX_Q_HEADS 128
#define RTP_MAX_INDEX_HEADS 32
#define RTP_MAX_HEADS_PER_INDEX_HEAD 16

typedef enum rtp_status {
  RTP_OK = 0,
  RTP_ERR_INVALID = 1,     /* bad argument */
  RTP_ERR_CAPACITY = 2,    /* a caller buffer is too small (lists, workspace) */
  RTP_ERR_UNSUPPORTED = 3, /* valid request this build does not implement */
  RTP_ERR_CUDA = 4,        /* a CUDA runtime call failed; see rtp_last_error */
  RTP_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out */
} rtp_status;

/* Opaque host-side context: device properties and the last error string. */
typedef struct rtp_ctx rtp_ctx;

/* Method parameters (Table 2 gives the paper's values: index_dim 16, top_p 0.9,
 * n_sink 4, window 8192).  The four head-map arrays are HOST pointers. */
typedef struct rtp_params {
  int32_t head_dim;      /* must be 128 */
  int32_t index_dim;     /* must be 16 */
  int32_t page_size;     /* must be 64 */
  int32_t n_q_heads;     /* <= RTP_MAX_Q_HEADS, multiple of n_kv_heads */
  int32_t n_kv_heads;
  int32_t n_index_heads; /* <= RTP_MAX_INDEX_HEADS */
  int32_t n_ret_q_heads; /* number of retrieval query heads */
  int32_t n_local_kv_heads;
  int32_t n_sink;        /* attention sinks of local heads (first n_sink tokens) */
  int32_t window;        /* sliding window of local heads: positions (m-window, m] */
  float top_p;           /* in (0, 1] */
  float score_scale;     /* temperature on the indexer score; 1.0 in the paper */
  float sm_scale;        /* softmax scale of the real attention, 1/sqrt(128) */
  const int32_t* ret_q_heads;          /* HOST [n_ret_q_heads] query-head ids */
  const int32_t* q_head_to_index_head; /* HOST [n_ret_q_heads] */
  const int32_t* index_head_kv;        /* HOST [n_index_heads] KV head of each index head */
  const int32_t* local_kv_heads;       /* HOST [n_local_kv_heads] */
  /* Selectable variants of the decode selection (row lists: rtp_topp_select with row arrays, rtp_sparse_attn_decode).
   * All zero = Eq. 5 as the paper states it.
   *   top_k > 0: the fixed-budget selector of Section 4.1 (k = 4096 there) instead of Top-P: the top_k keys with the
   *     largest indexer scores, equal scores going to the smaller position; every key when the row has fewer.  top_p is
   *     ignored; sel_mass then receives (keys taken) / (causal keys), not a softmax mass.
   *   force_sink / force_recent > 0: the first force_sink keys and the newest force_recent keys of the row (its own
   *     position included) are joined to the selected set whatever their scores.  They come after the regular entries
   *     of a list, sel_count counts them, sel_mass includes their softmax mass; sel_thresh / sel_tie_last still describe
   *     the regular rule alone.  force_sink + force_recent <= 65536.
   * The chunk (prefill) forms of the selection and the block-wise calls return RTP_ERR_UNSUPPORTED when any of the
   * three is set. */
  int32_t top_k;
  int32_t force_sink;
  int32_t force_recent;
} rtp_params;

/* Paged caches.  The index-key cache shares the KV block table. */
typedef struct rtp_cache {
  void* k_pages;              /* DEVICE bf16 [num_pages, n_kv_heads, 64, 128] */
  void* v_pages;              /* DEVICE bf16 [num_pages, n_kv_heads, 64, 128] */
  void* ikey_pages;           /* DEVICE bf16 [num_pages, n_index_heads, 64, 16]; see ikey_format */
  const int32_t* block_table; /* DEVICE int32 [batch, max_pages] physical page ids */
  const int32_t* seq_lens;    /* DEVICE int32 [batch] tokens present per sequence */
  int32_t num_pages;
  int32_t batch;
  int32_t max_pages;
  /* Optional: truncated cache for local heads (Sections 1 and 3.2: the full KV cache is kept for retrieval heads only).
   * When k_local_pages is not NULL,
   *   - k_pages / v_pages hold only the KV heads that are NOT in rtp_params.local_kv_heads, in increasing head order:
   *     bf16 [num_pages, n_kv_heads - n_local_kv_heads, 64, 128];
   *   - the local KV heads, in the order of rtp_params.local_kv_heads, live in
   *     k_local_pages / v_local_pages: bf16 [n_local_pages, n_local_kv_heads, 64, 128] behind their own table
   *     local_block_table: int32 [batch, sink_pages + ring_pages]: logical page p of a sequence is entry p for
   *     p < sink_pages and entry sink_pages + (p - sink_pages) % ring_pages otherwise, so a sequence holds its first
   *     sink_pages pages and its newest ring_pages pages.  sink_pages * 64 must cover n_sink; a call of rtp_local_attn
   *     needs ring_pages * 64 >= window + (tokens appended beyond the oldest row of the call) + 64;
   *   - rtp_kv_append writes every head to its pool (one call must not carry more than ring_pages * 64 tokens of a
   *     sequence: tokens of one call are written in no particular order); rtp_local_attn reads the local pool; the sparse and dense calls
   *     read the main pool (dense calls may then only name heads that live there).
   * All zero / NULL: one pool with every KV head (the layout above). */
  void* k_local_pages;
  void* v_local_pages;
  const int32_t* local_block_table;
  int32_t n_local_pages;
  int32_t sink_pages;
  int32_t ring_pages;
  /* Storage type of the index-key cache.  RTP_IKEY_BF16 (0): bf16, 32 bytes per token and index head.
   * RTP_IKEY_E4M3 (1): 8-bit floats (1 sign, 4 exponent, 3 mantissa bits, bias 7, largest magnitude 448, no
   * infinities), uint8 [num_pages, n_index_heads, 64, 16], 16 bytes per token and index head: half the bytes of the
   * decode scan.  rtp_index_keys then stores the fp32 projection rounded to the nearest E4M3 value (ties to even,
   * saturating); rtp_index_score and the row form of rtp_topp_select evaluate Eq. 4 on the decoded keys, with the
   * projected queries taken in fp16 (RTP_ERR_UNSUPPORTED in the status word if one exceeds 65504 in magnitude).  The
   * chunk form of rtp_topp_select, rtp_topp_select_blocks and the threshold form of rtp_sparse_attn_prefill need
   * the bf16 cache (RTP_ERR_UNSUPPORTED): the paper's method selects in decode only. */
  int32_t ikey_format;
} rtp_cache;

#define RTP_IKEY_BF16 0
#define RTP_IKEY_E4M3 1

/* ---- utility ------------------------------------------------------------ */

/* Library version, major*10000 + minor*100 + patch.  (No counterpart in the paper.) */
int32_t rtp_version(void);

/* Size in bytes of the two argument blocks as this library was compiled (what = 0: rtp_params, 1: rtp_cache; 0 for any
 * other value).  A binding that lays the blocks out itself compares them with its own before the first call. */
size_t rtp_struct_bytes(int32_t what);

/* Creates a context for the current CUDA device.  Returns RTP_ERR_CUDA when no
 * usable sm_100 device is current.  (No counterpart in the paper.) */
rtp_status rtp_create(rtp_ctx** out_ctx);
void rtp_destroy(rtp_ctx* ctx);

/* Text of the last error recorded on this context (never NULL). */
const char* rtp_last_error(const rtp_ctx* ctx);

/* Diagnostic hook for the bounded device-side waits (the paper has no counterpart).  Inside the tensor-core
 * kernels warps hand tiles to each other through barriers in shared memory; every such wait gives up after
 * `wait_limit_ns` nanoseconds (default two seconds), records RTP_ERR_TIMEOUT in the call's status word and the
 * kernel runs to its end without waiting again.  With drop_first_key_signal != 0 the key loader of the prefill
 * attention kernels withholds the signal for its first key tile, so that the next rtp_dense_attn_prefill /
 * rtp_local_attn / rtp_sparse_attn_prefill call on this context must report RTP_ERR_TIMEOUT (its output is
 * then undefined).  Pass (2000000000, 0) to restore the defaults.  Returns RTP_ERR_INVALID for a NULL context or
 * a limit <= 0. */
rtp_status rtp_debug_wait_test(rtp_ctx* ctx, int64_t wait_limit_ns, int32_t drop_first_key_signal);

/* Diagnostic hook for the decode selection (row form of rtp_topp_select).  It has two implementations with the same
 * results.  For contexts whose block table holds at most 36864 keys and calls of at most 2 x SM count (row, head) pairs
 * one CTA per pair keeps the row's scores in shared memory and runs the whole selection on them (up to 8192 keys it
 * also scores the keys itself; above, one kernel scores for all of them first): it is the faster one there.  Otherwise
 * the general path of several kernels over stored scores runs.  path = 1 forces the general path on this context,
 * path = 0 restores the choice above.  Returns RTP_ERR_INVALID for a NULL context or another value. */
rtp_status rtp_debug_select_path(rtp_ctx* ctx, int32_t path);

/* Bytes of DEVICE workspace that any call below needs for `rows` query rows
 * against sequences of at most `max_seq_len` tokens.  0 on invalid params.
 * The largest consumer is rtp_topp_select in chunk mode: a pool of 8 KB blocks
 * from which every (row, retrieval head) takes the space for the keys around
 * its cut on demand, sized at 32 KB per (row, head), rounded up to whole
 * tiles of 128 pairs (2 GB for 8192 rows x 8 heads).  A larger workspace is
 * used in full; a row that finds the pool empty narrows its candidates by one
 * more pass over the keys instead. */
size_t rtp_workspace_bytes(const rtp_params* params, int64_t rows, int64_t max_seq_len);

/* Synchronises `stream`, reads the DEVICE status word and returns it as an
 * rtp_status (RTP_ERR_CUDA if the stream reports an error). */
rtp_status rtp_check_status(rtp_ctx* ctx, const int32_t* status, void* stream);

/* ---- S0: index-key projection and cache append (Eq. 4, the W^K k_pre factor;
 *      Section 3.4 calls the result the "compressed K sequence") -------------
 * k_pre   DEVICE bf16 [T, n_index_heads, 128]  pre-RoPE keys of the index heads
 * w_k     DEVICE bf16 [n_index_heads, 128, 16]
 * tok_seq DEVICE int32 [T] sequence of each token; tok_pos DEVICE int32 [T] its position
 * Writes ikey_pages[block_table[seq][pos/64], j, pos%64, :] for every token and
 * index head j: fp32 accumulation, rounded to bf16.  Pages must already be
 * mapped in block_table.  Nothing else is written. */
rtp_status rtp_index_keys(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                          const void* k_pre, const void* w_k, const int32_t* tok_seq,
                          const int32_t* tok_pos, int64_t T, void* stream);

/* ---- cache append of new K/V rows (Section 3.2: the KV cache that prefill builds and decode
 *      extends; retrieval heads keep it whole) ------------------------------------
 * k_new, v_new DEVICE bf16 [T, n_kv_heads, 128] post-RoPE keys / values of T new tokens;
 * tok_seq, tok_pos DEVICE int32 [T].  Copies every row to
 * k_pages / v_pages[block_table[seq][pos/64], head, pos%64, :].  Tokens whose sequence or page
 * is out of range are skipped and RTP_ERR_INVALID is recorded in *status.  seq_lens is not
 * modified (it belongs to the caller). */
rtp_status rtp_kv_append(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                         const void* k_new, const void* v_new, const int32_t* tok_seq,
                         const int32_t* tok_pos, int64_t T, int32_t* status, void* stream);

/* ---- S1: query projection (Eq. 4, the W^Q q_pre factor) --------------------
 * q_pre  DEVICE bf16 [R, n_q_heads, 128] pre-RoPE queries (all heads; only the
 *        retrieval heads are read)
 * w_q    DEVICE bf16 [n_ret_q_heads, 128, 16]
 * qt_out DEVICE bf16 [R, n_ret_q_heads, 16]
 * The other calls project their queries themselves; this one returns the projection on its own, e.g. to
 * inspect or cache it. */
rtp_status rtp_index_queries(rtp_ctx* ctx, const rtp_params* params, const void* q_pre,
                             const void* w_q, int64_t R, void* qt_out, void* stream);

/* ---- S1-S3: indexer scores and softmax normaliser (Eq. 4; Section 3.3 for the
 *      distribution softmax(s) that top-p cuts) ------------------------------
 * Row i is the query at position row_pos[i] of sequence row_seq[i]; it scores
 * keys 0..row_pos[i] (inclusive).  DEVICE int32 row_seq, row_pos [R].
 * scores_out  DEVICE fp32 [R, n_ret_q_heads, score_stride] or NULL; entries past
 *             the row's last key are left untouched
 * row_max_out DEVICE fp32 [R, n_ret_q_heads] or NULL : M = max_n s
 * row_sum_out DEVICE fp32 [R, n_ret_q_heads] or NULL : Z = sum_n exp(s - M)
 * s = score_scale * sum_j qt_j kt_j with bf16 factors and fp32 accumulation. */
rtp_status rtp_index_score(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                           const void* q_pre, const void* w_q, const int32_t* row_seq,
                           const int32_t* row_pos, int64_t R, float* scores_out,
                           int64_t score_stride, float* row_max_out, float* row_sum_out,
                           void* workspace, size_t workspace_bytes, int32_t* status,
                           void* stream);

/* ---- S2-S4: fused indexer + top-p selection (Eq. 5, S = Top-P(s, p)) --------
 * Selects, per row and retrieval query head, the shortest prefix of the keys in
 * order of decreasing score (ties: smaller position first) whose softmax mass
 * reaches top_p.  Mass sums are fp32; a token whose cumulative mass before its
 * own inclusion is within 1e-5 of p may be included, and keys of exactly equal
 * score that straddle the cut are taken together when the whole group ends
 * within 5e-5 of p (both inside the 1e-4 band in which the set is free).  The
 * set is never empty; top_p == 1 selects every causal key.  Scores must be
 * finite and below 2^18 in magnitude, a chunk may reach at most position 2^21
 * (RTP_ERR_UNSUPPORTED otherwise).  The scores are always recomputed from the
 * index-key cache inside the kernels (16 dimensions cost less than reading a
 * materialised score back), so there is no scores-in variant.
 *
 * Rows: either DEVICE row_seq/row_pos [R] (any rows; the decode path), or
 * row_seq == row_pos == NULL and the rows are positions q_start..q_start+R-1 of
 * sequence seq_id (a prefill chunk).
 * sel_idx      DEVICE int32 [R, n_ret_q_heads, sel_stride] logical token
 *              positions in unspecified order, or NULL (thresholds only)
 * sel_count    DEVICE int32 [R, n_ret_q_heads] true size of the set, also when
 *              it exceeds sel_stride (then only sel_stride ids are written and
 *              RTP_ERR_CAPACITY is recorded in *status)
 * sel_mass     DEVICE fp32  [R, n_ret_q_heads] softmax mass of the set (fp32 estimate)
 * sel_thresh   DEVICE fp32  [R, n_ret_q_heads] smallest selected score
 * sel_tie_last DEVICE int32 [R, n_ret_q_heads] position bound for keys whose score
 *              equals sel_thresh: a key n belongs to the set iff s > thresh or
 *              (s == thresh and n <= tie_last).  Any value from the largest selected
 *              tied position up to (excluding) the smallest tied position left out
 *              describes the same set; the row's last position is returned when no
 *              tied key is left out.
 * status       DEVICE int32 [1] */
rtp_status rtp_topp_select(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                           const void* q_pre, const void* w_q, const int32_t* row_seq,
                           const int32_t* row_pos, int32_t seq_id, int32_t q_start, int64_t R,
                           int32_t* sel_idx, int64_t sel_stride, int32_t* sel_count,
                           float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                           int32_t* status, void* workspace, size_t workspace_bytes,
                           void* stream);

/* ---- S5 (+S8): sparse attention over selection lists (Eq. 5) ----------------
 * For every row and retrieval query head: softmax(q.k * sm_scale) over the listed
 * keys, times V; split over the list with a log-sum-exp merge when rows are few.
 * q    DEVICE bf16 [R, n_q_heads, 128] post-RoPE queries
 * out  DEVICE bf16 [R, n_q_heads, 128]; only retrieval heads' slots are written
 * lse  DEVICE fp32 [R, n_q_heads] natural-log-sum-exp of the scaled logits, or NULL
 * sel_idx / sel_count as written by rtp_topp_select (counts above sel_stride are
 * clamped).  Ids must be < the row's key count; others are skipped and
 * RTP_ERR_INVALID is recorded. */
rtp_status rtp_sparse_attn_decode(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                  const void* q, const int32_t* row_seq, const int32_t* row_pos,
                                  int64_t R, const int32_t* sel_idx, int64_t sel_stride,
                                  const int32_t* sel_count, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, int32_t* status,
                                  void* stream);

/* ---- rtp_sparse_attn_decode without a caller workspace (the paper has no counterpart; this is a
 *      packaging variant) -----------------------------------------------------------------
 * Same computation, arguments and results as rtp_sparse_attn_decode, for hosts that cannot provide
 * scratch memory at call time: e.g. a serving process whose device heap was handed over entirely to a
 * pool it does not own, a plugin that runs inside someone else's allocator-free region, or code that
 * runs where cudaMalloc is forbidden.  The split partials live in a fixed 512 KiB array that is part of
 * the library image (every GPU that loads the library holds it until the process exits); the call
 * allocates nothing and calls no allocating routine.
 *  - Limit: rows * n_ret_q_heads * n_splits * 520 bytes must fit in 512 KiB, where n_splits is the
 *    split count the library plans for the call (about 4 * SM count / (rows * heads), at most one
 *    split per 512 listed tokens, nothing at all for a single split; on a 148-SM device a decode
 *    batch of up to 63 sequences x 8 retrieval heads always fits).  Larger calls return RTP_ERR_CAPACITY before anything is launched
 *    and rtp_last_error says how many bytes were needed.
 *  - The first call on each device looks up the array's device address (once per device, with that
 *    device current); make that first call outside any CUDA stream capture.
 *  - All calls share the one array.  Nothing in it has to start at zero (every slot that is read was
 *    written earlier in the same call), and it keeps the last call's partials afterwards.  Two calls
 *    that overlap on the GPU (different streams, or graphs replayed concurrently) race on it: issue
 *    them in stream order, or use rtp_sparse_attn_decode with separate workspaces. */
rtp_status rtp_sparse_attn_decode_static(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                         const void* q, const int32_t* row_seq, const int32_t* row_pos,
                                         int64_t R, const int32_t* sel_idx, int64_t sel_stride,
                                         const int32_t* sel_count, void* out, float* lse, int32_t* status,
                                         void* stream);

/* ---- S6: sparse attention for a prefill chunk (Eq. 5 applied per query row; the
 *      paper itself keeps retrieval heads dense in prefill) -------------------
 * Rows are positions q_start..q_start+C-1 of sequence seq_id; causal.
 * With sel_idx != NULL the lists are used as in rtp_sparse_attn_decode.  With
 * sel_idx == NULL membership is re-evaluated inside the attention kernel from
 * (sel_thresh, sel_tie_last) and the indexer score, which needs q_pre and w_q:
 * the kernel visits every causal key tile of a row tile and masks the scores
 * of the keys outside each row's set (threshold-masked dense attention: with
 * one set per row and head the union over the 128 rows of a tile covers every
 * key tile, so there is nothing to skip).  This mode needs every query head of
 * a retrieval KV head to be a retrieval head on the same index head
 * (RTP_ERR_UNSUPPORTED otherwise).
 * q, q_pre DEVICE bf16 [C, n_q_heads, 128]; out/lse as above. */
rtp_status rtp_sparse_attn_prefill(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                   const void* q, const void* q_pre, const void* w_q,
                                   int32_t seq_id, int32_t q_start, int64_t C,
                                   const int32_t* sel_idx, int64_t sel_stride,
                                   const int32_t* sel_count, const float* sel_thresh,
                                   const int32_t* sel_tie_last, void* out, float* lse,
                                   void* workspace, size_t workspace_bytes, int32_t* status,
                                   void* stream);


/* ---- NEXT: block-wise top-p for prefill (Section 3.4) --------------------------------------------
 * The paper's kernel selects whole blocks of 64 keys rather than single tokens: every block of a row's indexer
 * scores is reduced to a log-sum-exp pair (m_b, l_b); blocks are taken in order of decreasing m_b (equal maxima:
 * the smaller block first) until their softmax mass, sum of l_b exp(m_b - M) / Z, reaches top_p.  Here a block is
 * one cache page, the order is exact (the paper deposits the pairs in a 256-bin histogram indexed by m_b; this
 * library resolves the bin in which the mass is reached down to single blocks), and the result is a bit per page.
 *
 * rtp_topp_select_blocks: rows are the C positions q_start .. q_start + C - 1 of sequence seq_id (a prefill chunk;
 * the chunk's index keys must have been appended).  q_pre: bf16 [C, n_q_heads, 128] device; w_q as in
 * rtp_topp_select.
 *   block_mask   uint32 [C, n_ret_q_heads, mask_words] device, written: bit (b & 31) of word b >> 5 of a row is set
 *                iff block b (keys 64 b .. 64 b + 63, cut at the row's own position) is selected.  Words beyond the
 *                row's last block are not written.  mask_words * 32 must cover ceil((q_start + C) / 64) blocks.
 *   sel_count    int32 [C, n_ret_q_heads]: number of selected blocks; sel_mass (may be NULL): their softmax mass;
 *   sel_thresh   (may be NULL): m_b of the last block taken (-inf when every block is taken);
 *   sel_tie_last (may be NULL): index of that block.
 *   workspace    device scratch of rtp_block_workspace_bytes(params, C, q_start + C) bytes.
 * Errors as rtp_topp_select; RTP_ERR_CAPACITY when mask_words or the workspace is too small.
 *
 * rtp_sparse_attn_prefill_blocks: exact attention of the retrieval heads' rows of the chunk over the keys of their
 * selected blocks (causal inside the row's last block); q: bf16 [C, n_q_heads, 128] post-RoPE; out / lse as
 * rtp_sparse_attn_prefill (retrieval heads' slots only).  Like the token-level call it needs every index head to
 * serve the whole query-head group of its KV head. */
size_t rtp_block_workspace_bytes(const rtp_params* params, int64_t rows, int64_t max_seq_len);
rtp_status rtp_topp_select_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                                  const void* w_q, int32_t seq_id, int32_t q_start, int64_t C, uint32_t* block_mask,
                                  int64_t mask_words, int32_t* sel_count, float* sel_mass, float* sel_thresh,
                                  int32_t* sel_tie_last, int32_t* status, void* workspace, size_t workspace_bytes,
                                  void* stream);
rtp_status rtp_sparse_attn_prefill_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                          int32_t seq_id, int32_t q_start, int64_t C, const uint32_t* block_mask,
                                          int64_t mask_words, void* out, float* lse, int32_t* status, void* stream);

/* The same block-wise rule for explicit rows (decode: the use Section 3.4 describes it for).
 * rtp_topp_select_blocks_rows: rows as in rtp_topp_select with row arrays.  For every (row, retrieval head) the
 *   selected blocks are written as LOGICAL page numbers (block b = keys 64 b .. 64 b + 63 of the row's sequence), in
 *   no particular order: block_idx DEVICE int32 [R, n_ret_q_heads, block_stride] (may be NULL: counts
 *   only), sel_count = number of blocks (a list longer than block_stride is cut and RTP_ERR_CAPACITY set in the status
 *   word), sel_mass = softmax mass of the selected blocks, sel_thresh = m_b of the last block taken, sel_tie_last = its
 *   block number (-inf / last block when every block is taken).  At most 16384 blocks per row (RTP_ERR_UNSUPPORTED
 *   beyond; max_pages of the cache is what counts).  Workspace: rtp_block_workspace_bytes(params, R, max_seq_len).
 *   Works on bf16 and 8-bit index keys.  The selectable variants of rtp_params (top_k, forced positions) are for token
 *   lists: RTP_ERR_UNSUPPORTED here.
 * rtp_sparse_attn_decode_blocks: exact attention of every retrieval query head over the keys of its listed pages
 *   (the positions of the row's last page beyond the row's own are left out), split-KV with LSE merge as
 *   rtp_sparse_attn_decode; block_count as written by the selection; a page number outside the row's causal pages sets
 *   RTP_ERR_INVALID in the status word and is skipped.  With a workspace of rtp_workspace_bytes(params, R,
 *   max_seq_len) the lists of the query heads that share a KV head are first merged into their union (Section 3.2:
 *   what a KV head must supply is the union of its heads' sets) and the group is attended in one pass over it, every
 *   head seeing only its own pages: pages that several heads selected are read once.  With a smaller (or no)
 *   workspace every head gathers its own pages; the results are the same. */
rtp_status rtp_topp_select_blocks_rows(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q_pre,
                                       const void* w_q, const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                                       int32_t* block_idx, int64_t block_stride, int32_t* sel_count, float* sel_mass,
                                       float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* workspace,
                                       size_t workspace_bytes, void* stream);
rtp_status rtp_sparse_attn_decode_blocks(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache, const void* q,
                                         const int32_t* row_seq, const int32_t* row_pos, int64_t R,
                                         const int32_t* block_idx, int64_t block_stride, const int32_t* block_count,
                                         void* out, float* lse, void* workspace, size_t workspace_bytes,
                                         int32_t* status, void* stream);

/* ---- S7: local heads, attention sinks + sliding window (Section 3.2, Table 2) -
 * Row at position m attends to {n <= m : n < n_sink or n > m - window}.
 * Rows as in rtp_topp_select (row arrays = decode path with split-KV; NULL
 * arrays = prefill chunk seq_id, q_start).  Only the query heads of
 * params->local_kv_heads are computed and written. */
rtp_status rtp_local_attn(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                          const void* q, const int32_t* row_seq, const int32_t* row_pos,
                          int32_t seq_id, int32_t q_start, int64_t R, void* out, float* lse,
                          void* workspace, size_t workspace_bytes, int32_t* status,
                          void* stream);

/* ---- S9: dense causal attention, the in-library comparator (what retrieval
 *      heads run during the paper's prefill, Section 3.2) ---------------------
 * kv_heads HOST int32 [n_heads] KV heads whose query heads are computed; NULL =
 * all heads.  rtp_dense_attn_prefill: rows q_start.. of seq_id;
 * rtp_dense_attn_decode: rows given by DEVICE row_seq/row_pos, split-KV. */
rtp_status rtp_dense_attn_prefill(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                  const void* q, int32_t seq_id, int32_t q_start, int64_t C,
                                  const int32_t* kv_heads, int32_t n_heads, void* out, float* lse,
                                  int32_t* status, void* stream);
rtp_status rtp_dense_attn_decode(rtp_ctx* ctx, const rtp_params* params, const rtp_cache* cache,
                                 const void* q, const int32_t* row_seq, const int32_t* row_pos,
                                 int64_t R, const int32_t* kv_heads, int32_t n_heads, void* out,
                                 float* lse, void* workspace, size_t workspace_bytes,
                                 int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RTP_H_ */
