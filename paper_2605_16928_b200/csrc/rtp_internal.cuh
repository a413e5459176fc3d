// Internal declarations shared by the kernels and the C-ABI layer (sm_100a only).
#pragma once

#include <utility>

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "rtp.h"

namespace rtp {

constexpr int kHeadDim = RTP_HEAD_DIM;     // 128
constexpr int kIndexDim = RTP_INDEX_DIM;   // 16
constexpr int kPage = RTP_PAGE_SIZE;       // 64
constexpr int kPageShift = 6;

// Selection (decode-style) constants.
constexpr int kCandCap = 4096;             // boundary candidates resolved exactly per (row, head)
constexpr float kMassMargin = 1e-5f;       // relative slack added to p*Z against fp32 summation error

// Head maps, passed to kernels by value.
struct HeadMaps {
  uint8_t ret_q_head[RTP_MAX_Q_HEADS];      // query-head id of retrieval head i
  uint8_t q2ih[RTP_MAX_Q_HEADS];            // index head of retrieval head i
  uint8_t slot_in_ih[RTP_MAX_Q_HEADS];      // position of retrieval head i inside its index head's list
  uint8_t ih_kv[RTP_MAX_INDEX_HEADS];       // KV head of index head j
  uint8_t ih_nheads[RTP_MAX_INDEX_HEADS];   // number of retrieval heads scoring against index head j
  uint8_t ih_heads[RTP_MAX_INDEX_HEADS][RTP_MAX_HEADS_PER_INDEX_HEAD];
  uint8_t kv_list[RTP_MAX_Q_HEADS];         // KV heads processed by a local / dense call
  int32_t n_kv_list;
  // Query heads a local call computes but does not write: the retrieval heads inside a KV group that is otherwise
  // local (a mixed group, Section 3.2: the head partition is over query heads).  Bit q of word q / 32.
  uint32_t skip_q[RTP_MAX_Q_HEADS / 32];
  __host__ __device__ bool skips(int qh) const { return (skip_q[qh >> 5] >> (qh & 31)) & 1u; }
};

struct CacheView {
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* ikey;
  const int32_t* block_table;
  const int32_t* seq_lens;
  int32_t num_pages, batch, max_pages;
  int32_t n_kv, n_ih;      // n_kv: KV heads per page of the pool k / v point to
  // A view of one pool.  cap_tokens: logical capacity of a sequence (the main block table's pages), used wherever a
  // length is clamped.  ring_pages > 0: block_table has sink_pages + ring_pages entries per sequence and logical
  // page p >= sink_pages lives in entry sink_pages + (p - sink_pages) % ring_pages.  kv_slot[h]: position of KV head h
  // inside a page of this pool (0xff: the head is not stored here).
  int32_t cap_tokens, sink_pages, ring_pages;
  uint8_t kv_slot[32];
  // != 0: the index-key cache holds 8-bit floats (E4M3), 16 bytes per token and index head, instead of bf16
  int32_t ikey_fp8;
};

struct Dims {
  int32_t n_q, n_kv, n_ih, n_ret, group;
  int32_t n_sink, window;
  float top_p, score_scale, sm_scale;
  int32_t top_k;                       // > 0: the fixed-budget selector (Section 4.1) in the decode selection
  int32_t force_sink, force_recent;    // positions joined to every selected set of the decode selection
  // bounded device-side waits give up after this many nanoseconds; wait_test != 0: the key loader of the prefill
  // attention kernel withholds the signal for its first tile (rtp_debug_wait_test)
  unsigned long long wait_ns;
  int32_t wait_test;
  int32_t select_path;   // decode selection: 0 = one CTA per (row, head) where the context is short enough, 1 = always the general path
};

// Rows of a call: explicit arrays (decode) or a contiguous chunk of one sequence.
struct Rows {
  const int32_t* seq;   // may be NULL
  const int32_t* pos;   // may be NULL
  int32_t seq_id, q_start;
  int64_t R;
  __device__ __forceinline__ int row_seq(int64_t r) const { return seq ? seq[r] : seq_id; }
  __device__ __forceinline__ int row_pos(int64_t r) const { return pos ? pos[r] : q_start + (int)r; }
};

// Per (row, retrieval head) selection state kept in the workspace between passes.
struct SelState {
  uint32_t max_key;      // ordered key of the row maximum (atomicMax during the first pass)
  uint32_t lo_key;       // current bucket [lo_key, hi_key] of ordered keys that holds the threshold
  uint32_t hi_key;
  uint32_t span;         // hi_key - lo_key + 1
  int32_t shift;         // key levels: bin = (key - lo_key) >> shift, in [0, 64)
  int32_t mode;          // 0 = refining, 1 = collect candidates, 2 = select all, 3 = exact ties (scan)
  float M;               // row maximum
  float Z;               // sum exp(s - M)
  float target;          // mass to reach, relative to M (p * Z * (1 + margin))
  float mass_above;      // mass of keys above the bucket
  float ref_s;           // key levels: masses are accumulated relative to exp(ref_s - M)
  float e_ref;           // exp(ref_s - M)
  int32_t cnt_above;     // number of keys above the bucket (counted by the compaction pass)
  int32_t bucket_cnt;    // keys inside the bucket (exact after a key level)
  int32_t emit_cnt;      // ids written by the compaction pass
  int32_t cand_cnt;      // candidates written by the compaction pass
  int32_t n_keys;        // causal key count of the row
  int32_t pad;
};

enum SelMode { kRefine = 0, kCollect = 1, kSelectAll = 2, kTieScan = 3 };

// A function attribute such as the dynamic shared memory limit is a per-device setting: it is applied the first time
// a kernel is launched on each device (one bit per device ordinal; safe to call from several threads).
struct PerDeviceOnce {
  std::atomic<uint64_t> bits[4] = {};
};
template <class Kernel>
inline cudaError_t set_dyn_smem_once(Kernel kernel, int bytes, PerDeviceOnce& once, bool max_carveout = false) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 256) return cudaErrorInvalidDevice;
  const uint64_t bit = 1ull << (dev & 63);
  if (once.bits[dev >> 6].load(std::memory_order_acquire) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  if (max_carveout) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) return e;
  }
  once.bits[dev >> 6].fetch_or(bit, std::memory_order_release);
  return cudaSuccess;
}

// Launch of a kernel of the decode chain (see chain_wait in rtp_device.cuh): the kernel may overlap the tail and the
// launch latency of the kernel before it in the stream.
template <class... KArgs, class... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// SM count of the current device (queried once per device; `fallback` when no device can be asked, e.g. when only
// sizes are computed on a host without a GPU).
inline int current_sm_count(int fallback) {
  static std::atomic<int> cache[256] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 256) {
    cudaGetLastError();
    return fallback;
  }
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return fallback;
  }
  cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

// ---- host launchers (one per .cu file) ---------------------------------------
cudaError_t launch_index_keys(const CacheView& cv, const Dims& d, const __nv_bfloat16* k_pre,
                              const __nv_bfloat16* w_k, const int32_t* tok_seq, const int32_t* tok_pos,
                              int64_t T, cudaStream_t st);
cudaError_t launch_kv_append(const CacheView& cv, int n_src_heads, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new,
                             const int32_t* tok_seq, const int32_t* tok_pos, int64_t T, int32_t* status,
                             cudaStream_t st);
cudaError_t launch_index_queries(const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q_pre,
                                 const __nv_bfloat16* w_q, int64_t R, __nv_bfloat16* qt, cudaStream_t st);

size_t score_workspace_bytes(const Dims& d, int64_t R, int64_t max_len, int sm_count);
cudaError_t launch_index_score(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const __nv_bfloat16* qt, int64_t max_len, float* scores, int64_t score_stride,
                               float* row_max, float* row_sum, void* ws, int32_t* status, int sm_count,
                               cudaStream_t st);

size_t select_rows_workspace_bytes(const Dims& d, int64_t R, int64_t max_len);
cudaError_t launch_select_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const __nv_bfloat16* qt, int64_t max_len, int32_t* sel_idx, int64_t sel_stride,
                               int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                               int32_t* status, void* ws, int sm_count, cudaStream_t st);

size_t select_chunk_workspace_bytes(const Dims& d, const HeadMaps& hm, int64_t R);
cudaError_t launch_select_chunk(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride,
                                int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                int32_t* status, void* ws, size_t ws_bytes, int sm_count, cudaStream_t st);

// kSetPages: like kSetList, but the list holds logical page numbers and every listed page is taken whole
// kSetUnion: one list per (row, KV head): the union of the pages its query heads selected, every entry a page number
//            (low 24 bits) with one flag bit per query head of the group (bit 24 + g: head g selected the page); the
//            whole group is attended in one pass over the union (GQA packing), a head sees only its own pages
enum AttnSet { kSetList = 0, kSetLocal = 1, kSetDense = 2, kSetPages = 3, kSetUnion = 4 };
size_t attn_rows_workspace_bytes(const Dims& d, int64_t R, int n_units, int group, int sm_count, int64_t max_len);
cudaError_t launch_attn_rows(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows, int set,
                             const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                             const int32_t* sel_count, __nv_bfloat16* out, float* lse, void* ws,
                             size_t ws_bytes, int64_t max_len, int32_t* status, int sm_count, cudaStream_t st);

size_t attn_rows_static_scratch_bytes();
cudaError_t launch_attn_rows_static(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                    const __nv_bfloat16* q, const int32_t* sel_idx, int64_t sel_stride,
                                    const int32_t* sel_count, __nv_bfloat16* out, float* lse, int64_t max_len,
                                    int32_t* status, int sm_count, size_t* needed_bytes, cudaStream_t st);

enum PrefillMode { kPrefillDense = 0, kPrefillLocal = 1, kPrefillSparse = 2, kPrefillBlocks = 3 };
cudaError_t launch_attn_prefill(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                const __nv_bfloat16* q, const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start,
                                int64_t C, const float* sel_thresh, const int32_t* sel_tie_last,
                                __nv_bfloat16* out, float* lse, int32_t* status, int sm_count, cudaStream_t st,
                                const uint32_t* blk_mask = nullptr, int64_t mask_words = 0);

cudaError_t launch_attn_prefill_tc(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                   const __nv_bfloat16* q, const __nv_bfloat16* qt, const float* sel_thresh,
                                   const int32_t* sel_tie_last, int32_t seq_id, int32_t q_start, int64_t C,
                                   __nv_bfloat16* out, float* lse, int32_t* status, cudaStream_t st,
                                   const uint32_t* blk_mask, int64_t mask_words);

// Block-wise top-p of a prefill chunk (Section 3.4): one bit per (row, retrieval head, page).
size_t select_blocks_workspace_bytes(const Dims& d, const HeadMaps& hm, int64_t R, int64_t max_len, int sm_count);
size_t select_rows_blocks_workspace_bytes(const Dims& d, int64_t R, int64_t max_len);
size_t block_union_bytes(const Dims& d, int64_t R, int64_t max_len);
// Page lists per retrieval head -> one flagged list per (row, KV head of hm.kv_list); ws holds block_union_bytes.
cudaError_t launch_block_union(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                               const int32_t* blk_idx, int64_t blk_stride, const int32_t* blk_cnt, int64_t max_len,
                               void* ws, int32_t** uni_idx, int64_t* uni_stride, int32_t** uni_cnt, int32_t* status,
                               cudaStream_t st);
cudaError_t launch_select_rows_blocks(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                      const __nv_bfloat16* qt, int64_t max_len, int32_t* blk_idx, int64_t blk_stride,
                                      int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                      int32_t* status, void* ws, int sm_count, cudaStream_t st);
cudaError_t launch_select_blocks(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                 const __nv_bfloat16* qt, uint32_t* mask, int64_t mask_words, int32_t* sel_count,
                                 float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* ws,
                                 size_t ws_bytes, int sm_count, cudaStream_t st);

}  // namespace rtp
