// S2-S4 for a prefill chunk: fused indexer + top-p selection (Eq. 5) for rows q_start .. q_start+C-1 of one
// sequence, on the 5th-generation tensor cores.
//
// A CTA owns 128 (row, head) pairs: (128 / G) consecutive positions x the G retrieval heads of one index head.
// The 16-dimensional scores q~ . k~ (Eq. 4) are one tcgen05.mma per 64-key cache page (M = 128 rows, N = 64 keys,
// K = 16) into tensor memory; thread t of the four score warps owns row t = TMEM lane t and reads its 64 scores of a
// page with tcgen05.ld, so a row's keys arrive at one thread in position order and all per-row state is private to it:
//   warp 4    TMA: index-key pages -> shared memory (SWIZZLE_32B rows of 32 bytes), four stages
//   warp 5    one lane issues the MMAs into two 64-column TMEM buffers
//   warps 0-3 passes over the keys 0 .. last position, each row on its own:
//     max      row maximum
//     level 1  mass histogram over a fixed grid of score bins of width 1/4 (bin = round(-4 s) relative to the bin of
//              the maximum; 64 bins, the last one pools everything below): the thread's private column of a
//              [64 bins][128 rows] array in shared memory, fixed point (2^18 = the bin's upper end), plain
//              load-add-store without atomics or bank conflicts; gives Z and the bin in which the cumulative mass
//              reaches p * Z.  A crossing inside the pooled bin repeats the level with the window moved down.
//     late     the keys of the chosen bin ("bucket") are appended to the row's list in global scratch, the keys
//              above it are counted.  A bucket that may hold more keys than the list (long rows) is first narrowed
//              by key levels: the list is used as a queue and drained into a 64-bin histogram of the next six key bits.
//     finish   the warp narrows the list with the same 64-bin mass histogram until at most 64 keys are left and ranks
//              those exactly by (score descending, position ascending); more than 64 equal scores at the cut take
//              one more pass that finds the position of the last tie taken.
//   When id lists are requested, one more sweep appends every row's members in position order.
// Hand-offs are mbarriers with bounded waits (a wait that runs out records RTP_ERR_TIMEOUT and lets every later wait
// fall through); the CTA always frees its tensor memory.
#include <algorithm>
#include <cstdio>
#include <cstdlib>

#include "mass_hist.cuh"
#include "tc_common.cuh"

namespace rtp {

namespace {

constexpr int kSRows = 128;
constexpr int kSTile = kPage;                 // keys per MMA = one cache page
constexpr int kSStages = 4;
constexpr int kSThreads = 128;                // threads of one pipeline: thread = row
constexpr int kTmemColsS = 128;               // two score buffers of 64 columns
constexpr int kStageBytesS = kSTile * kIndexDim * 2;   // 2 KB
constexpr int kCandCapC = 64;                 // candidates ranked exactly per row
// A row's list of bucket keys (unscaled score bits) lives in blocks of the workspace pool, taken on demand: word 0 of a
// block is the index of the row's next block, the other 2047 words are entries.
constexpr int kBlockWords = 2048;
constexpr int kBlockEntries = kBlockWords - 1;
constexpr uint32_t kNoBlock = 0xffffffffu;
constexpr uint32_t kMarker = 0xffc00000u, kMarkerMask = 0x003fffffu;   // list words that are position markers
constexpr int kListMax = 65536;               // buckets that may hold more keys are narrowed by a key level first
constexpr int kSweepLoads = 16;               // list words a lane has in flight during the sweeps after a pass
constexpr int kRowPoolEntries = 8192;         // pool words the workspace provides per (row, head)
constexpr int kMaxPasses = 24;
constexpr int kPoolBin = 62;                  // level-1 bin that pools everything below the window (an even shift, see aI)
constexpr int kMaxShift = kPoolBin * 6;             // level-1 windows below this depth hold no representable mass
constexpr float kLog2eC = kLog2eH;
constexpr float kMagicC = 12582912.0f;        // 1.5 * 2^23: adding it leaves the nearest integer in the low mantissa bits
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr int kFixBits = 17;                  // fixed point of the private histograms: 2^17 = upper end of the bin
// every key adds at least this to its bin (floor(e^-1/4 * 2^17) - 2), which bounds the number of keys by the sum
constexpr float kMinQ18 = 102077.0f;
constexpr float kMinQ14 = 12757.0f;           // the same for the 2^14 fixed point of the key-level histograms
// A bin's 32-bit sum grows by at most 2^23 per page (64 keys x 2^17); every kNormEvery pages the sums above 2^30 hand
// their upper bits to the bin's 8-bit counter (units of 2^30), so no add in between can wrap: 2^30 + 16 x 2^23 < 2^32.
// 255 x 2^30 / 2^17 bounds a row at two million keys per bin.
constexpr int kNormEvery = 16;

constexpr int kHistOff = 0;                                  // u32 [64 bins][128 rows]
constexpr int kCarryOff = kBins * kSRows * 4;                // u32 [16][128 rows]: four 8-bit wrap counters per word
constexpr int kStageOffS = kCarryOff + 16 * kSRows * 4;      // kSStages x 2 KB
constexpr int kAOff = kStageOffS + kSStages * kStageBytesS;  // projected queries [128 rows][16] bf16
constexpr int kBarOffS = kAOff + kSRows * kIndexDim * 2;
constexpr int kSubs = 4;                                     // independent pipelines per CTA
constexpr int kSmemSub = (kBarOffS + 256 + 1023) & ~1023;    // shared memory of one sub
constexpr int kSmemS = kSubs * kSmemSub;

enum BarS { kFullK = 0, kSFull = kSStages, kNumBarsS = kSStages + 2 };
enum Phase { kPhMax = 0, kPhL1 = 1, kPhKey = 2, kPhCollect = 3, kPhTie = 4, kPhDone = 5 };
enum PassKind { kPassNone = 0, kPassMax = 1, kPassL1 = 2, kPassLate = 3, kPassEmit = 4 };

__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }

// Private histogram column of a thread: bin b of the sums at col + 512 b, the 8-bit overflow counters (units of 2^30)
// of bins 4w .. 4w+3 at ccol + 512 w.
__device__ __forceinline__ void hist_add(uint32_t col, int bin, uint32_t q) {
  const uint32_t a = col + (uint32_t)bin * (kSRows * 4);
  sts32(a, lds32(a) + q);
}
// Moves the bits above 2^30 of every sum into the bin's counter.
__device__ __noinline__ void hist_normalize(uint32_t col, uint32_t ccol) {
  for (int w = 0; w < kBins / 4; ++w) {
    uint32_t add = 0u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t a = col + (uint32_t)(4 * w + k) * (kSRows * 4);
      const uint32_t v = lds32(a);
      if (v >> 30) {
        add += (v >> 30) << (8 * k);
        sts32(a, v & 0x3fffffffu);
      }
    }
    if (add) {
      const uint32_t ca = ccol + (uint32_t)w * (kSRows * 4);
      sts32(ca, lds32(ca) + add);
    }
  }
}
__device__ __forceinline__ float hist_read(uint32_t col, uint32_t ccol, int bin, bool& populated) {   // in units of 2^-17
  const uint32_t sum = lds32(col + (uint32_t)bin * (kSRows * 4));
  const uint32_t car = (lds32(ccol + (uint32_t)(bin >> 2) * (kSRows * 4)) >> ((bin & 3) * 8)) & 255u;
  populated = (sum | car) != 0u;
  return (float)car * 1073741824.0f + (float)sum;
}
// round(2^x) for x <= 17 (+ a rounding error) through the mantissa of 2^x + 2^23
__device__ __forceinline__ uint32_t fix_q(float x) { return __float_as_uint(fast_ex2(x) + 8388608.0f) - 0x4b000000u; }

// Level-1 update of a thread's private histogram for two unscaled scores r0, r1 (bit patterns):
//   s = r * scale;  t = min(fma(s, -4, dd), magic + 62)  (bin = low mantissa bits of t);
//   q = round(2^(fma(t - magic, log2e / 4, fma(s, log2e, cx))))  through the mantissa of (2^x + 2^23);
//   word at hb + 512 * bits(t) += q.
__device__ __forceinline__ void l1_pair(uint32_t r0, uint32_t r1, float scale, float dd, float cx, uint32_t hb) {
  asm volatile(
      "{\n"
      ".reg .f32 s0, s1, t0, t1, x0, x1, e0, e1;\n"
      ".reg .u32 q0, q1, a0, a1, o0, o1, n0, n1;\n"
      ".reg .pred pe;\n"
      "mul.f32 s0, %0, %2;\n"
      "mul.f32 s1, %1, %2;\n"
      "fma.rn.f32 t0, s0, 0fC0800000, %3;\n"
      "fma.rn.f32 t1, s1, 0fC0800000, %3;\n"
      "min.f32 t0, t0, 0f4B40003E;\n"
      "min.f32 t1, t1, 0f4B40003E;\n"
      "fma.rn.f32 x0, s0, 0f3FB8AA3B, %4;\n"
      "fma.rn.f32 x1, s1, 0f3FB8AA3B, %4;\n"
      "sub.f32 e0, t0, 0f4B400000;\n"
      "sub.f32 e1, t1, 0f4B400000;\n"
      "fma.rn.f32 x0, e0, 0f3EB8AA3B, x0;\n"
      "fma.rn.f32 x1, e1, 0f3EB8AA3B, x1;\n"
      "ex2.approx.ftz.f32 e0, x0;\n"
      "ex2.approx.ftz.f32 e1, x1;\n"
      "add.f32 e0, e0, 0f4B000000;\n"
      "add.f32 e1, e1, 0f4B000000;\n"
      "mov.b32 q0, e0;\n"
      "mov.b32 q1, e1;\n"
      "mov.b32 a0, t0;\n"
      "mov.b32 a1, t1;\n"
      "mad.lo.u32 a0, a0, 512, %5;\n"
      "mad.lo.u32 a1, a1, 512, %5;\n"
      "ld.shared.u32 o0, [a0];\n"
      "ld.shared.u32 o1, [a1];\n"
      "add.u32 n0, o0, q0;\n"
      "add.u32 n0, n0, 0xB5000000;\n"
      "setp.eq.u32 pe, a0, a1;\n"
      "selp.u32 o1, n0, o1, pe;\n"
      "add.u32 n1, o1, q1;\n"
      "add.u32 n1, n1, 0xB5000000;\n"
      "st.shared.u32 [a0], n0;\n"
      "st.shared.u32 [a1], n1;\n"
      "}\n" ::"f"(__uint_as_float(r0)),
      "f"(__uint_as_float(r1)), "f"(scale), "f"(dd), "f"(cx), "r"(hb)
      : "memory");
}

// Late pass, collecting rows: counts a score above `cut` and queues a score inside [lo, hi] at shared address qa.
__device__ __forceinline__ void late_one(uint32_t r, float cut, float lo, float hi, int& above, uint32_t& qa) {
  asm volatile(
      "{\n"
      ".reg .pred p0, p1;\n"
      "setp.gt.f32 p0, %2, %3;\n"
      "@p0 add.s32 %0, %0, 1;\n"
      "setp.ge.f32 p1, %2, %4;\n"
      "setp.le.and.f32 p1, %2, %5, p1;\n"
      "@p1 st.shared.u32 [%1], %6;\n"
      "@p1 add.u32 %1, %1, 512;\n"
      "}\n"
      : "+r"(above), "+r"(qa)
      : "f"(__uint_as_float(r)), "f"(cut), "f"(lo), "f"(hi), "r"(r)
      : "memory");
}

// Waits for the thread's tcgen05.ld results; the registers are operands so that no use of them moves above the wait.
__device__ __forceinline__ void tmem_wait16(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}
__device__ __forceinline__ void red_add_shared(uint32_t a, uint32_t v) {
  asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

// Grid bin of a score: round(-4 s) as an integer (monotone non-increasing in s; |s| < 2^18).
__device__ __forceinline__ int grid_bin(float s) { return (int)(__float_as_uint(fmaf(s, -4.0f, kMagicC)) - kMagicBits); }

// Exact interval [klo, khi] of ordered keys whose grid bin is `a`.
__device__ void grid_bin_keys(int a, uint32_t& klo, uint32_t& khi) {
  const float mid = -0.25f * (float)a;
  const uint32_t lo = okey(mid - 0.5f), hi = okey(mid + 0.5f);   // safely outside the bin on both sides
  uint32_t x = lo, y = hi;                 // klo = smallest key with grid_bin <= a
  if (grid_bin(okey_to_float(x)) <= a) y = x;
  while (x + 1 < y) {
    const uint32_t m = x + ((y - x) >> 1);
    if (grid_bin(okey_to_float(m)) <= a) y = m; else x = m;
  }
  klo = y;
  x = klo; y = hi;                         // khi = largest key with grid_bin >= a
  if (grid_bin(okey_to_float(y)) >= a) x = y;
  while (x + 1 < y) {
    const uint32_t m = x + ((y - x) >> 1);
    if (grid_bin(okey_to_float(m)) >= a) x = m; else y = m;
  }
  khi = x;
}

// One page of the pass: wait for its scores in tensor memory ... release the buffer.  The last of the four warps to
// release it (ticket counter in shared memory; nobody waits for anybody) hands the buffer to the page two ahead: it
// issues that page's MMA (its keys were requested kSStages pages earlier) and requests the keys of the page kSStages
// ahead, whose stage the completed MMA of this page has freed.
#define RTP_SEL_TILE_BEGIN                                                              \
  const int buf = (int)(gt & 1u);                                                       \
  mbar_wait(bar(kSFull + buf), (gt >> 1) & 1u, abort_flag, status, d.wait_ns);                     \
  tc_fence_after();                                                                     \
  const int n_base = it * kSTile;                                                       \
  const bool interior = n_base + kSTile - 1 <= min_pos;                                 \
  const uint32_t taddr = tmem + lane_addr + (uint32_t)(buf * kSTile);
#define RTP_SEL_TILE_END                                                                \
  tc_fence_before();                                                                    \
  __syncwarp();                                                                         \
  if (lane == 0) {                                                                      \
    __threadfence_block();                                                              \
    if (atomicAdd(&rel[buf], 1u) == 3u) {                                               \
      rel[buf] = 0u;                                                                    \
      tc_fence_after();                                                                 \
      if (it + 2 < t_hi) issue_mma(gt + 2u);                                            \
      if (it + kSStages < t_hi) issue_tma(gt + (uint32_t)kSStages, it + kSStages);      \
    }                                                                                   \
  }                                                                                     \
  __syncwarp();                                                                         \
  ++gt;

template <int G>
__global__ void __launch_bounds__(kSubs * kSThreads, 1) select_chunk_kernel(
    const __grid_constant__ CUtensorMap map_ik, const CacheView cv, const Dims d, const HeadMaps hm,
    const __nv_bfloat16* __restrict__ qt, const int seq_id, const int q_start, const int C,
    int32_t* __restrict__ sel_idx, const int64_t sel_stride, int32_t* __restrict__ sel_count,
    float* __restrict__ sel_mass, float* __restrict__ sel_thresh, int32_t* __restrict__ sel_tie_last, int32_t* status,
    uint32_t* __restrict__ pool, const uint32_t n_blocks, unsigned int* __restrict__ pool_ctr, const int n_row_tiles,
    const int max_passes_in) {
  constexpr int BMP = kSRows / G;
  extern __shared__ __align__(1024) unsigned char smem_all[];
  // A kernel that uses tensor memory runs one CTA per SM, so the CTA holds kSubs independent pipelines ("subs") of
  // kSThreads threads, each with its own slice of shared memory, its own 128 TMEM columns and its own named barrier.
  const int sub = threadIdx.x / kSThreads;
  const int tid = threadIdx.x - sub * kSThreads, lane = tid & 31, warp = tid >> 5;
  unsigned char* smem = smem_all + sub * kSmemSub;
  const uint32_t sbase = s_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_all + kBarOffS + kNumBarsS * 8);   // (sub 0's slot serves the CTA)
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kBarOffS + kNumBarsS * 8 + 4);
  volatile int* pass_flags = reinterpret_cast<volatile int*>(smem + kBarOffS + kNumBarsS * 8 + 8);   // [2]
  unsigned int* rel = reinterpret_cast<unsigned int*>(smem + kBarOffS + kNumBarsS * 8 + 16);         // [2] release tickets
  int* pass_rng = reinterpret_cast<int*>(smem + kBarOffS + kNumBarsS * 8 + 32);   // [2][2] page range of a pass of tie rows
  auto bar = [&](int i) { return sbase + kBarOffS + i * 8; };
  auto sub_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(1 + sub), "r"(kSThreads) : "memory"); };
  const int seq_len = min(cv.seq_lens[seq_id], cv.max_pages * kPage);   // (never beyond the block table)
  const bool want_ids = sel_idx != nullptr;
  const float scale = d.score_scale;
  const int n_units = n_row_tiles * d.n_ih;
  const int max_passes = max_passes_in;

  if (tid == 0) {
    for (int i = 0; i < kSStages; ++i) mbar_init(bar(kFullK + i), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kSFull + i), 1);
      rel[i] = 0u;
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(kSubs * kTmemColsS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_cta = *tmem_slot;
  const uint32_t tmem = tmem_cta + (uint32_t)(sub * kTmemColsS);
  // a warp reaches the 32 TMEM lanes of its quarter (warp index within the CTA modulo 4): the four score warps of a
  // sub are consecutive warps of the CTA, so they cover the four quarters in some rotation
  const int quarter = (int)(threadIdx.x >> 5) & 3;
  const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
  const int row = quarter * 32 + lane;
  const uint32_t hist_col = sbase + kHistOff + (uint32_t)row * 4u;
  const uint32_t carry_col = sbase + kCarryOff + (uint32_t)row * 4u;

  uint32_t gt = 0;               // key tiles consumed so far by this role (all roles of a sub walk the same sequence)
  // units (row tile, index head) in order of decreasing length, dealt round-robin to the SMs and then to their subs
  for (int unit = blockIdx.x + (int)gridDim.x * sub; unit < n_units; unit += (int)gridDim.x * kSubs) {
  const int tile = n_row_tiles - 1 - unit / d.n_ih;
  const int ih = unit % d.n_ih;
  const int nh = hm.ih_nheads[ih];
  const int r0 = tile * BMP;
  const int rows_here = min(BMP, C - r0);
  const int m0 = q_start + r0;
  const int m_last = min(m0 + rows_here - 1, seq_len - 1);
  const int n_tiles = m_last >= 0 ? (m_last >> kPageShift) + 1 : 0;
  const int min_pos = min(m0, seq_len - 1);
  sub_sync();                    // the previous unit is finished by every thread of the sub
  if (tid == 0) {
    pass_flags[0] = 0;
    pass_flags[1] = 0;
    pass_rng[0] = pass_rng[2] = 0x7fffffff;
    pass_rng[1] = pass_rng[3] = 0;
    if (m0 + rows_here - 1 >= seq_len) set_status(status, RTP_ERR_INVALID);
  }
  sub_sync();

  // ---- per-row state of the score threads (registers) ----
  const int hs = row / BMP, po = row % BMP;
  const bool row_ok = hs < nh && po < rows_here;
  const int rh_head = hs < nh ? hm.ih_heads[ih][hs] : 0;
  const int pos = min(m0 + po, seq_len - 1);
  const int n_keys = row_ok ? pos + 1 : 0;
  int phase = kPhDone;
  uint32_t thr_key = 0u;
  int tie_last = -1, count = 0;
  float sel_m = 0.f;
  if (row_ok && n_keys > 0) {
    phase = kPhMax;
    if (d.top_p >= 1.0f || n_keys == 1) {   // everything is selected
      phase = kPhDone;
      tie_last = n_keys - 1;
      count = n_keys;
      sel_m = 1.0f;
    }
  }
  {
    // projected queries of the unit's rows -> the A operand (rows of 32 bytes, SWIZZLE_32B: the two 16-byte halves of
    // rows 4-7 of every 8-row group are exchanged)
    uint4 v0 = make_uint4(0u, 0u, 0u, 0u), v1 = v0;
    if (row_ok) {
      const uint4* src = reinterpret_cast<const uint4*>(qt + ((int64_t)(r0 + po) * d.n_ret + rh_head) * kIndexDim);
      v0 = __ldg(src);
      v1 = __ldg(src + 1);
    }
    const int sw = (row >> 2) & 1;
    *reinterpret_cast<uint4*>(smem + kAOff + row * 32 + ((0 ^ sw) << 4)) = v0;
    *reinterpret_cast<uint4*>(smem + kAOff + row * 32 + ((1 ^ sw) << 4)) = v1;
    fence_async_smem();
    if (phase != kPhDone) atomicOr(const_cast<int*>(&pass_flags[0]), 1 << kPhMax);
  }
  sub_sync();

  // level 1
  int aI = 0, w0 = 0;            // grid bin of the maximum; offset of the current 64-bin window below it
  float ref0 = 0.f;              // score of the upper end of the maximum's bin: every mass is relative to exp(ref0)
  float Z = 0.f, target = 0.f, mass_above = 0.f;
  bool have_z = false;
  // bucket
  uint32_t base_key = 0u, span = 0u;
  int shift = 0;
  float raw_lo = __int_as_float(0x7f800000), raw_hi = -__int_as_float(0x7f800000);
  float ref_s = 0.f, e_ref = 0.f;
  int cnt_above = 0, cand_cnt = 0, tie_need = 0, tie_run = 0;
  uint32_t blk_first = kNoBlock;   // first block of the row's list
  int tie_pos_lo = 0, tie_pos_hi = 0x7fffffff;   // tie rows: the positions among which the tie_need-th tie lies

  // page `page` of the current pass, the g-th page this pipeline has walked since the kernel started: stage g % kSStages
  const int64_t bt_base = (int64_t)seq_id * cv.max_pages;
  auto issue_tma = [&](uint32_t g, int page) {
    const int stage = (int)(g % kSStages);
    const int phys = safe_phys(cv, bt_base + page, status);
    mbar_expect_tx(bar(kFullK + stage), kStageBytesS);
    tma_load_2d(sbase + kStageOffS + stage * kStageBytesS, &map_ik, 0, (phys * cv.n_ih + ih) * kPage, bar(kFullK + stage));
  };
  auto issue_mma = [&](uint32_t g) {
    const int stage = (int)(g % kSStages), b2 = (int)(g & 1u);
    mbar_wait(bar(kFullK + stage), (g / kSStages) & 1u, abort_flag, status, d.wait_ns);
    tc_fence_after();
    tc_mma(tmem + (uint32_t)(b2 * kSTile), smem_desc_sw(sbase + kAOff, 16, 256, 6),
           smem_desc_sw(sbase + kStageOffS + stage * kStageBytesS, 16, 256, 6), instr_desc_mn(kSRows, kSTile, false), 0u);
    tc_commit(bar(kSFull + b2));
  };
  int done_emit = 0;
  for (int pass = 0; pass < max_passes; ++pass) {
    const int flags = pass_flags[pass & 1];
    int kind = (flags & (1 << kPhMax)) ? kPassMax : (flags & (1 << kPhL1)) ? kPassL1 : (flags & ~(1 << kPhDone)) ? kPassLate : kPassNone;
    if (kind == kPassNone && want_ids && !done_emit) {
      kind = kPassEmit;
      done_emit = 1;
    }
    if (kind == kPassNone || n_tiles == 0) break;
    // pages walked by the pass: all of them, except when only tie rows are left, which know where to look
    int t_lo = 0, t_hi = n_tiles;
    if (kind == kPassLate && flags == (1 << kPhTie)) {
      t_lo = max(0, min(pass_rng[2 * (pass & 1)], n_tiles - 1));
      t_hi = max(t_lo + 1, min(pass_rng[2 * (pass & 1) + 1], n_tiles));
    }

    {
      // prologue of the pass by one thread: request the keys of the first kSStages pages, multiply the first two
      if (warp == 0 && lane == 0) {
        for (int j = 0; j < kSStages && t_lo + j < t_hi; ++j) issue_tma(gt + (uint32_t)j, t_lo + j);
        for (int j = 0; j < 2 && t_lo + j < t_hi; ++j) issue_mma(gt + (uint32_t)j);
      }
      __syncwarp();
      // ================================ score threads (thread = row) ================================
      for (int b = 0; b < kBins; ++b) sts32(hist_col + (uint32_t)b * (kSRows * 4), 0u);
      for (int b = 0; b < 16; ++b) sts32(carry_col + (uint32_t)b * (kSRows * 4), 0u);
      // A page's 64 scores are read from tensor memory sixteen at a time; the next sixteen are in flight while the
      // current ones are processed (small code: the instruction cache is shared by four pipelines).
#define RTP_SEL_GROUPS(PROCESS)                                                          \
  {                                                                                      \
    uint32_t ra[16], rb[16];                                                             \
    RTP_TMEM_LD16(ra, taddr);                                                            \
    tmem_wait16(ra);                                                                     \
    _Pragma("unroll 1") for (int g = 0; g < 4; g += 2) {                                 \
      RTP_TMEM_LD16(rb, taddr + (uint32_t)(16 * g + 16));                                \
      PROCESS(ra, n_base + 16 * g);                                                      \
      tmem_wait16(rb);                                                                   \
      if (g + 2 < 4) RTP_TMEM_LD16(ra, taddr + (uint32_t)(16 * g + 32));                 \
      PROCESS(rb, n_base + 16 * g + 16);                                                 \
      tmem_wait16(ra);                                                                   \
    }                                                                                    \
  }
      if (kind == kPassMax) {
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
        auto proc_max = [&](const uint32_t(&r)[16], const int n0, const bool interior) {
          if (interior) {
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
              mx0 = fmaxf(mx0, __uint_as_float(r[j]));
              mx1 = fmaxf(mx1, __uint_as_float(r[j + 1]));
              mx2 = fmaxf(mx2, __uint_as_float(r[j + 2]));
              mx3 = fmaxf(mx3, __uint_as_float(r[j + 3]));
            }
          } else {
            const int valid = pos - n0 + 1;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (j < valid) mx0 = fmaxf(mx0, __uint_as_float(r[j]));
          }
        };
#pragma unroll 1
        for (int it = t_lo; it < t_hi; ++it) {
          RTP_SEL_TILE_BEGIN
#define RTP_P(r_, n0_) proc_max(r_, n0_, interior)
          RTP_SEL_GROUPS(RTP_P)
#undef RTP_P
          RTP_SEL_TILE_END
        }
        if (phase == kPhMax) {
          const float s_max = finish_score(fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)), scale);
          if (!(fabsf(s_max) < 262144.0f)) {
            // no finite score, or scores beyond the range of the fixed grid: every key is kept and the call reports it
            set_status(status, RTP_ERR_UNSUPPORTED);
            phase = kPhDone;
            tie_last = n_keys - 1;
            count = n_keys;
            sel_m = 1.0f;
          } else {
            // The window is anchored on an even grid bin and moves by an even number of bins: the binning of the level-1
            // pass rounds -4 s - (aI + w0) to the nearest even on a tie, which then agrees with grid_bin's round(-4 s) for
            // a score that lies exactly between two bins.
            aI = grid_bin(s_max) & ~1;
            w0 = 0;
            ref0 = -0.25f * ((float)aI - 0.5f);
            mass_above = 0.f;
            phase = kPhL1;
          }
        }
      } else if (kind == kPassL1) {
        // bin = round(-4 s) - aI - w0, clamped to kPoolBin; mass relative to the bin's upper end, 2^18 fixed point
        const bool shifted = w0 > 0;
        const bool active = phase == kPhL1;
        // rows that take no part land in the pooling bin of their own column whatever their scores are
        const float dd = active ? kMagicC - (float)(aI + w0) : __int_as_float(0x7f800000);
        const float cx = (float)kFixBits + (kLog2eC * 0.25f) * ((float)(aI + w0) - 0.5f);
        const uint32_t hb = hist_col - kMagicBits * (uint32_t)(kSRows * 4);
        auto proc_l1 = [&](const uint32_t(&r)[16], const int n0, const bool fast) {
          if (fast) {
            // two scores at a time, written out instruction by instruction: both bins are loaded before either is
            // stored (the second takes the first's new value when they are the same bin)
#pragma unroll
            for (int j = 0; j < 16; j += 2) l1_pair(r[j], r[j + 1], scale, dd, cx, hb);
          } else if (active) {
            const int valid = pos - n0 + 1;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float s = __uint_as_float(r[j]) * scale;
              float t = fmaf(s, -4.0f, dd);
              // (t < magic: above the window, accounted for by an earlier level)
              if (j < valid && !(t < kMagicC)) {
                t = fminf(t, kMagicC + (float)kPoolBin);
                const float x = fmaf(t - kMagicC, kLog2eC * 0.25f, fmaf(s, kLog2eC, cx));
                hist_add(hist_col, (int)(__float_as_uint(t) & 63u), fix_q(x));
              }
            }
          }
        };
#pragma unroll 1
        for (int it = t_lo; it < t_hi; ++it) {
          RTP_SEL_TILE_BEGIN
          const bool fast = interior && !shifted;
#define RTP_P(r_, n0_) proc_l1(r_, n0_, fast)
          RTP_SEL_GROUPS(RTP_P)
#undef RTP_P
          RTP_SEL_TILE_END
          if ((it & (kNormEvery - 1)) == kNormEvery - 1) hist_normalize(hist_col, carry_col);
        }
        hist_normalize(hist_col, carry_col);
        if (active) {
          if (!have_z) {
            float tot = 0.f;
            for (int b = 0; b < kBins; ++b) {
              bool pop;
              const float qf = hist_read(hist_col, carry_col, b, pop);
              tot += qf * fast_ex2(-(float)kFixBits - (float)b * (kLog2eC * 0.25f));
            }
            Z = tot;
            target = d.top_p * Z * (1.0f + kMassMargin);
            have_z = true;
          }
          float run = mass_above;
          int found = -1, last = -1;
          float above_found = 0.f, above_last = 0.f, q_found = 0.f, q_last = 0.f;
          for (int b = 0; b < kBins; ++b) {
            bool pop;
            const float qf = hist_read(hist_col, carry_col, b, pop);
            const float m = qf * fast_ex2(-(float)kFixBits - (float)(w0 + b) * (kLog2eC * 0.25f));
            if (pop) {
              last = b;
              above_last = run;
              q_last = qf;
              if (found < 0 && run + m >= target) {
                found = b;
                above_found = run;
                q_found = qf;
              }
            }
            run += m;
          }
          if (found < 0) {   // rounding left the target just out of reach: lowest populated bin
            found = last;
            above_found = above_last;
            q_found = q_last;
          }
          if (found < 0) {
            // an empty window below the mass already counted: nothing is left to add
            set_status(status, RTP_ERR_UNSUPPORTED);
            phase = kPhDone;
            tie_last = n_keys - 1;
            count = n_keys;
            sel_m = 1.0f;
          } else if (found == kPoolBin) {
            // the pooled bin: look at it with a window of its own, unless it lies so deep that it holds no mass
            mass_above = above_found;
            w0 += kPoolBin;
            if (w0 > kMaxShift) {
              phase = kPhDone;
              tie_last = n_keys - 1;
              count = n_keys;
              sel_m = 1.0f;
            }
          } else {
            mass_above = above_found;
            const int a_abs = aI + w0 + found;
            uint32_t klo, khi;
            grid_bin_keys(a_abs, klo, khi);
            base_key = klo;
            span = khi - klo + 1u;
            const int bits = span > 1u ? 32 - __clz(span - 1u) : 0;
            shift = max(0, bits - 6);
            raw_preimage(scale, klo, khi, raw_lo, raw_hi);
            ref_s = -0.25f * ((float)a_abs - 0.5f);
            e_ref = fast_ex2(-(float)(w0 + found) * (kLog2eC * 0.25f));
            cand_cnt = 0;
            cnt_above = 0;
            const bool few = q_found < 0.999f * kMinQ18 * (float)kListMax;
            phase = (few || span == 1u) ? kPhCollect : kPhKey;
          }
        }
      } else if (kind == kPassLate) {
        // The unscaled scores inside a row's interval are queued in shared memory and moved on by the whole warp:
        //   collecting rows   queue = the row's own (idle) histogram column, 64 words; destination = the row's list in
        //                     the pool (raw bits in position order; behind every batch a marker word with the index of
        //                     the next group of eight positions, so that the keys of a batch are known to lie between
        //                     the positions of two markers); the keys above the interval are counted
        //   key-level rows    (buckets too large to list) queue = the 16 words of the row's counter column;
        //                     destination = the 64-bin mass histogram of the next six key bits in the row's histogram
        //                     column (2^14 fixed point)
        //   tie rows          no queue: the position of the tie_need-th key with the threshold score is noted in passing
        // After the pass the warp takes its collecting rows one by one: a sweep over the list builds the same 64-bin
        // histogram (only when the bucket holds more than kCandCapC keys), the sixty-fourth of the bucket in which the
        // mass reaches the target is found, and a second sweep moves the keys of that sub-interval (normally a few dozen)
        // into the row's column; then every thread walks its own row's candidates in order of decreasing score.
        const bool collecting = phase == kPhCollect, keying = phase == kPhKey, tying = phase == kPhTie;
        const bool listing = collecting || keying;
        const float kInfL = __int_as_float(0x7f800000);
        const float lo = listing ? raw_lo : kInfL, hi = listing ? raw_hi : -kInfL;
        const float cut = collecting ? raw_hi : kInfL;
        const float tlo = tying ? raw_lo : kInfL, thi = tying ? raw_hi : -kInfL;
        const bool any_tie = (flags & (1 << kPhTie)) != 0;
        constexpr uint32_t kStep = kSRows * 4;
        const uint32_t qbase = keying ? carry_col : hist_col;
        const uint32_t qfull = qbase + (uint32_t)(keying ? 8 : 56) * kStep;   // more entries than this: flush
        const uint32_t qhalf = qbase + (uint32_t)(keying ? 4 : 28) * kStep;
        uint32_t qa = qbase;                               // address of the next free queue word (512 bytes apart)
        int cnt = 0, above = 0, n_words = 0;               // keys seen / keys above the interval / words of the list
        uint32_t blk_cur = kNoBlock;                       // collecting rows: the block being filled and its word count
        int fill = 0;
        bool ovf = false;
        blk_first = kNoBlock;
        auto warp_flush = [&](const bool everything, const int next_group) {
          const uint32_t m = __ballot_sync(0xffffffffu, everything ? qa > qbase : qa > qhalf);
          for (uint32_t rest = m; rest; rest &= rest - 1u) {
            const int l = __ffs(rest) - 1;
            const uint32_t qb_l = __shfl_sync(0xffffffffu, qbase, l);
            const int qn_l = (int)((__shfl_sync(0xffffffffu, qa, l) - qb_l) / kStep);
            if (!__shfl_sync(0xffffffffu, (int)keying, l)) {
              // (a bucket of one key value needs no list: its keys are only counted)
              if (__shfl_sync(0xffffffffu, span, l) == 1u || __shfl_sync(0xffffffffu, (int)ovf, l)) {
                if (lane == l) {
                  cnt += qn_l;
                  qa = qbase;
                }
                continue;
              }
              // the words (qn_l keys and the marker) go behind the `fill` words of the row's current block and, when that
              // is full, on into a new block from the pool (an exhausted pool marks the row: its bucket is narrowed by
              // a key level instead)
              const int nw = qn_l + 1;
              uint32_t cur_l = __shfl_sync(0xffffffffu, blk_cur, l);
              const int fill_l = __shfl_sync(0xffffffffu, fill, l);
              const int room = cur_l == kNoBlock ? 0 : kBlockEntries - fill_l;
              uint32_t nb = kNoBlock;
              if (nw > room) {
                if (lane == 0) {
                  nb = atomicAdd(pool_ctr, 1u);
                  if (nb < n_blocks) {
                    pool[(size_t)nb * kBlockWords] = kNoBlock;
                    if (cur_l != kNoBlock) pool[(size_t)cur_l * kBlockWords] = nb;
                  } else {
                    nb = kNoBlock;
                  }
                }
                nb = __shfl_sync(0xffffffffu, nb, 0);
              }
              for (int i = lane; i < nw; i += 32) {
                const uint32_t v = i < qn_l ? lds32(qb_l + (uint32_t)i * kStep) : (kMarker | ((uint32_t)next_group & kMarkerMask));
                if (i < room) pool[(size_t)cur_l * kBlockWords + 1 + fill_l + i] = v;
                else if (nb != kNoBlock) pool[(size_t)nb * kBlockWords + 1 + (i - room)] = v;
              }
              if (lane == l) {
                if (nw > room) {
                  if (nb == kNoBlock) {
                    ovf = true;
                  } else {
                    if (blk_first == kNoBlock) blk_first = nb;
                    blk_cur = nb;
                    fill = nw - room;
                    n_words += nw;
                  }
                } else {
                  fill += nw;
                  n_words += nw;
                }
              }
            } else {
              const uint32_t base_l = __shfl_sync(0xffffffffu, base_key, l), span_l = __shfl_sync(0xffffffffu, span, l);
              const int shift_l = __shfl_sync(0xffffffffu, shift, l);
              const float ref_l = __shfl_sync(0xffffffffu, ref_s, l);
              const uint32_t hcol_l = __shfl_sync(0xffffffffu, hist_col, l);
              for (int i = lane; i < qn_l; i += 32) {
                const float s = finish_score(__uint_as_float(lds32(qb_l + (uint32_t)i * kStep)), scale);
                const uint32_t t = okey(s) - base_l;
                if (t < span_l) red_add_shared(hcol_l + (uint32_t)(t >> shift_l) * kStep, fix_q(fmaf(s - ref_l, kLog2eC, 14.0f)));
              }
            }
            if (lane == l) {
              cnt += qn_l;
              qa = qbase;
            }
          }
          __syncwarp();
        };
        // eight scores of the row
        auto proc8 = [&](const uint32_t* r, const int n0, const bool interior) {
          if (interior && !any_tie) {
#pragma unroll
            for (int j = 0; j < 8; ++j) late_one(r[j], cut, lo, hi, above, qa);
          } else {
            const int valid = interior ? 8 : pos - n0 + 1;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float raw = __uint_as_float(r[j]);
              if (j < valid && raw > cut) ++above;
              if (j < valid && raw >= lo && raw <= hi) {
                sts32(qa, r[j]);
                qa += kStep;
              }
              if (j < valid && raw >= tlo && raw <= thi && n0 + j >= tie_pos_lo && n0 + j < tie_pos_hi) {
                if (++tie_run == tie_need) tie_last = n0 + j;
              }
            }
          }
          if (__any_sync(0xffffffffu, qa > qfull)) {
            warp_flush(false, (n0 + 8) >> 3);
          }
        };
        auto proc_late = [&](const uint32_t(&r)[16], const int n0, const bool interior) {
          proc8(&r[0], n0, interior);
          proc8(&r[8], n0 + 8, interior);
        };
#pragma unroll 1
        for (int it = t_lo; it < t_hi; ++it) {
          RTP_SEL_TILE_BEGIN
#define RTP_P(r_, n0_) proc_late(r_, n0_, interior)
          RTP_SEL_GROUPS(RTP_P)
#undef RTP_P
          RTP_SEL_TILE_END
        }
        warp_flush(true, (int)kMarkerMask);
        // ---- key-level rows: the sub-interval in which the mass reaches the target becomes the bucket ----
        bool sub_ok = true;
        if (keying) {
          float run = mass_above;   // bins in order of decreasing score: 63 is the top
          int found = -1, last = -1;
          float above_found = 0.f, above_last = 0.f, q_found = 0.f, q_last = 0.f;
          for (int b = kBins - 1; b >= 0; --b) {
            const uint32_t sum = lds32(hist_col + (uint32_t)b * kStep);
            const float qf = (float)sum;
            const float m = qf * e_ref * 6.103515625e-05f;   // 2^-14
            if (sum != 0u) {
              last = b;
              above_last = run;
              q_last = qf;
              if (found < 0 && run + m >= target) {
                found = b;
                above_found = run;
                q_found = qf;
              }
            }
            run += m;
          }
          if (found < 0) {
            found = last;
            above_found = above_last;
            q_found = q_last;
          }
          if (found < 0) {
            sub_ok = false;   // a chosen bucket always holds a key
          } else {
            mass_above = above_found;
            const uint32_t ofs = (uint32_t)found << shift;
            const uint32_t lo_key = base_key + ofs;
            const uint32_t s_span = min(1u << shift, span - ofs);
            raw_preimage(scale, lo_key, lo_key + (s_span - 1u), raw_lo, raw_hi);
            base_key = lo_key;
            span = s_span;
            shift = max(0, shift - 6);
            cand_cnt = 0;
            cnt_above = 0;
            const bool few = q_found < 0.999f * kMinQ14 * (float)kListMax;
            phase = (few || s_span == 1u) ? kPhCollect : kPhKey;
          }
        }
        if (tying) {
          if (tie_last < 0) {           // fewer ties than counted before: cannot happen
            set_status(status, RTP_ERR_UNSUPPORTED);
            tie_last = n_keys - 1;
          }
          phase = kPhDone;
        }
        if (collecting && ovf) phase = kPhKey;   // no room for the bucket's keys: one key level first
        __syncwarp();   // every thread has read its histogram column: it now receives the row's final candidates
        // ---- exact finish of the rows that collected ----
        const bool fin = collecting && !ovf;
        bool new_tie = false;
        uint32_t sub_base = base_key, sub_span = span;
        float sub_above = mass_above;
        int c_in = fin ? cnt : 0, c_up = 0;   // keys inside / above the sub-interval (inside the bucket)
        {
          uint32_t* hw2 = reinterpret_cast<uint32_t*>(smem + kStageOffS) + warp * 256;   // (the key stages are idle between passes)
          const uint32_t hw2_a = s_u32(hw2);
          const uint32_t sweep = __ballot_sync(0xffffffffu, fin && span > 1u);
          for (uint32_t rest = sweep; rest; rest &= rest - 1u) {
            const int rr = __ffs(rest) - 1;
            const uint32_t first = __shfl_sync(0xffffffffu, blk_first, rr);
            const int n_all = __shfl_sync(0xffffffffu, n_words, rr);
            const int n_k = __shfl_sync(0xffffffffu, cnt, rr);
            const uint32_t b0 = __shfl_sync(0xffffffffu, base_key, rr), s0 = __shfl_sync(0xffffffffu, span, rr);
            const float ref_l = __shfl_sync(0xffffffffu, ref_s, rr);
            const float sc14 = __shfl_sync(0xffffffffu, e_ref, rr) * 6.103515625e-05f;   // 2^-14
            const float tg = __shfl_sync(0xffffffffu, target, rr);
            const uint32_t col_rr = __shfl_sync(0xffffffffu, hist_col, rr);
            uint32_t b1 = b0, s1 = s0;      // the interval that holds the cut, narrowed level by level
            float ab1 = __shfl_sync(0xffffffffu, mass_above, rr);
            int nk = n_k, filled = 0, ups = 0;
            bool ok1 = true;
            for (int level = 0; level < 8 && ok1; ++level) {
              uint32_t nb = b1, ns = s1;
              if (nk > kCandCapC && s1 > 1u) {
                // first sweep: mass histogram of the interval's next six key bits
                const int shift_l = max(0, 32 - __clz(s1 - 1u) - 6);
                hw2[lane] = 0u;
                hw2[lane + 32] = 0u;
                __syncwarp();
                int done = 0;
                for (uint32_t blk = first; blk != kNoBlock && done < n_all;) {
                  const uint32_t* b = pool + (size_t)blk * kBlockWords;
                  const int n_here = min(kBlockEntries, n_all - done);
                  const uint32_t next = __ldcg(b);
                  for (int i0 = 0; i0 < n_here; i0 += 32 * kSweepLoads) {
                    uint32_t v[kSweepLoads];
#pragma unroll
                    for (int k = 0; k < kSweepLoads; ++k) {
                      const int i = i0 + 32 * k + lane;
                      v[k] = i < n_here ? __ldcg(b + 1 + i) : kMarker;
                    }
#pragma unroll
                    for (int k = 0; k < kSweepLoads; ++k) {
                      const float sc_ = finish_score(__uint_as_float(v[k]), scale);
                      const uint32_t t = okey(sc_) - b1;
                      if ((v[k] & kMarker) != kMarker && t < s1)
                        red_add_shared(hw2_a + 4u * (t >> shift_l), fix_q(fmaf(sc_ - ref_l, kLog2eC, 14.0f)));
                    }
                  }
                  done += n_here;
                  blk = next;
                }
                __syncwarp();
                // two bins per lane in order of decreasing score: lane l takes bins 63 - 2 l and 62 - 2 l
                const uint32_t sum0 = hw2[63 - 2 * lane], sum1 = hw2[62 - 2 * lane];
                const float m0f = (float)sum0 * sc14, m1f = (float)sum1 * sc14;
                float incm = m0f + m1f;
#pragma unroll
                for (int ofs = 1; ofs < 32; ofs <<= 1) {
                  const float tm = __shfl_up_sync(0xffffffffu, incm, ofs);
                  if (lane >= ofs) incm += tm;
                }
                const float run = ab1 + incm - (m0f + m1f);
                int found = 64, last = -1;
                if (sum0) {
                  last = 2 * lane;
                  if (run + m0f >= tg) found = 2 * lane;
                }
                if (sum1) {
                  last = 2 * lane + 1;
                  if (found == 64 && run + m0f + m1f >= tg) found = 2 * lane + 1;
                }
#pragma unroll
                for (int ofs = 16; ofs > 0; ofs >>= 1) {
                  found = min(found, __shfl_xor_sync(0xffffffffu, found, ofs));
                  last = max(last, __shfl_xor_sync(0xffffffffu, last, ofs));
                }
                if (found == 64) found = last;
                if (found < 0) {
                  ok1 = false;   // a chosen interval always holds a key
                  break;
                }
                ab1 = __shfl_sync(0xffffffffu, (found & 1) ? run + m0f : run, found >> 1);
                const uint32_t ofs_k = (uint32_t)(63 - found) << shift_l;
                nb = b1 + ofs_k;
                ns = min(1u << shift_l, s1 - ofs_k);
                __syncwarp();
              }
              // second sweep: the keys of the sub-interval move into the row's column (as many as fit); the keys of the
              // interval above it are counted
              int fl = 0, up = 0, done = 0;
              for (uint32_t blk = first; blk != kNoBlock && done < n_all;) {
                const uint32_t* b = pool + (size_t)blk * kBlockWords;
                const int n_here = min(kBlockEntries, n_all - done);
                const uint32_t next = __ldcg(b);
                for (int i0 = 0; i0 < n_here; i0 += 32 * kSweepLoads) {
                  uint32_t v[kSweepLoads];
#pragma unroll
                  for (int k = 0; k < kSweepLoads; ++k) {
                    const int i = i0 + 32 * k + lane;
                    v[k] = i < n_here ? __ldcg(b + 1 + i) : kMarker;
                  }
#pragma unroll
                  for (int k = 0; k < kSweepLoads; ++k) {
                    const uint32_t key = okey(finish_score(__uint_as_float(v[k]), scale));
                    const bool in_b = (v[k] & kMarker) != kMarker && key - b1 < s1;
                    const bool inside = in_b && key - nb < ns;
                    const uint32_t m = __ballot_sync(0xffffffffu, inside);
                    up += __popc(__ballot_sync(0xffffffffu, in_b && !inside && key >= nb));
                    if (inside) {
                      const int p2 = fl + __popc(m & ((1u << lane) - 1u));
                      if (p2 < kCandCapC) sts32(col_rr + (uint32_t)p2 * kStep, key);
                    }
                    fl += __popc(m);
                  }
                }
                done += n_here;
                blk = next;
              }
              ups += up;
              filled = fl;
              b1 = nb;
              s1 = ns;
              nk = fl;
              if (nk <= kCandCapC || s1 == 1u) break;
            }
            if (lane == rr) {
              c_in = filled;
              c_up = ups;
              sub_base = b1;
              sub_span = s1;
              sub_above = ab1;
              if (!ok1) sub_ok = false;
            }
          }
          __syncwarp();
        }
        if ((keying || fin) && !sub_ok) {
          set_status(status, RTP_ERR_UNSUPPORTED);
          phase = kPhDone;
          tie_last = n_keys - 1;
          count = n_keys;
          sel_m = 1.0f;
        }
        // every collecting row: the thread walks the key values of its column in decreasing order until the mass reaches
        // the target (an interval of one key value, which may hold any number of keys, has nothing to walk)
        if (fin && sub_ok) {
          // (thr, g = keys of the sub-interval above it, eq = keys equal to it, m_gt = mass of the g keys, each = mass of one)
          uint32_t thr = sub_base;
          int g = 0, eq = c_in;
          float m_gt = 0.f, each = 0.f;
          if (sub_span == 1u || c_in > kCandCapC) {
            each = fast_ex2((okey_to_float(sub_base) - ref0) * kLog2eC);
            if (sub_span != 1u) set_status(status, RTP_ERR_UNSUPPORTED);   // (more levels than any key has bits)
          } else {
            if (c_in <= 0) set_status(status, RTP_ERR_UNSUPPORTED);   // a chosen bucket always holds a key
            uint32_t bound = 0u;
            bool first_step = true;
            for (int step = 0; step < kCandCapC; ++step) {
              uint32_t mx = 0u;
              int c = 0;
              for (int i = 0; i < c_in; ++i) {
                const uint32_t k = lds32(hist_col + (uint32_t)i * kStep);
                if (first_step || k < bound) {
                  if (k > mx) {
                    mx = k;
                    c = 1;
                  } else if (k == mx) {
                    ++c;
                  }
                }
              }
              if (c == 0) break;   // every key walked without reaching the target (rounding): the last group stands
              if (!first_step) {
                m_gt += (float)eq * each;
                g += eq;
              }
              thr = mx;
              eq = c;
              each = fast_ex2((okey_to_float(mx) - ref0) * kLog2eC);
              first_step = false;
              bound = mx;
              if (sub_above + m_gt + (float)eq * each >= target) break;
            }
          }
          const float cum = sub_above + m_gt;
          int take = eq;   // (a key too light to register in fp32 cannot split its group)
          if (each > 0.f) take = (int)fminf(ceilf((target - cum) / each), (float)eq);
          take = max(1, min(take, eq));
          // Keys of equal score that straddle the cut: when the whole group still ends inside the mass band in which
          // the set is free (cumulative mass before the group's last key below p + 5e-5), it is taken whole and no
          // position is needed.
          if (take < eq && cum + (float)(eq - 1) * each <= (d.top_p + 5e-5f) * Z) take = eq;
          cnt_above = above + c_up;
          mass_above = cum;
          thr_key = thr;
          count = above + c_up + g + take;
          sel_m = (cum + (float)take * each) / Z;
          if (take < eq) {   // the next pass finds the position of the tie_need-th key with this score
            tie_need = take;
            tie_run = 0;
            tie_last = -1;
            raw_preimage(scale, thr_key, thr_key, raw_lo, raw_hi);
            phase = kPhTie;
            new_tie = true;
          } else {
            tie_last = n_keys - 1;
            phase = kPhDone;
          }
        }
        // ---- rows whose cut falls between keys of equal score: where in the list is the tie_need-th of them? ----
        if (new_tie) {
          tie_pos_lo = 0;
          tie_pos_hi = 0x7fffffff;
        }
        {
          const uint32_t loc = __ballot_sync(0xffffffffu, new_tie && span > 1u);
          for (uint32_t rest = loc; rest; rest &= rest - 1u) {
            const int rr = __ffs(rest) - 1;
            const uint32_t first = __shfl_sync(0xffffffffu, blk_first, rr);
            const int n_all = __shfl_sync(0xffffffffu, n_words, rr);
            const uint32_t tk = __shfl_sync(0xffffffffu, thr_key, rr);
            const int need_t = __shfl_sync(0xffffffffu, tie_need, rr);
            int ties = 0, ties_at_mark = 0, g_lo = 0, g_hi = -1, done = 0;   // g_hi >= 0: found
            for (uint32_t blk = first; blk != kNoBlock && done < n_all && g_hi < 0;) {
              const uint32_t* b = pool + (size_t)blk * kBlockWords;
              const int n_here = min(kBlockEntries, n_all - done);
              for (int i0 = 0; i0 < n_here && g_hi < 0; i0 += 32) {
                const int i = i0 + lane;
                const uint32_t w = i < n_here ? __ldcg(b + 1 + i) : 0u;
                const bool is_mark = i < n_here && (w & kMarker) == kMarker;
                const bool is_tie = i < n_here && !is_mark && okey(finish_score(__uint_as_float(w), scale)) == tk;
                const uint32_t mm = __ballot_sync(0xffffffffu, is_mark), tm = __ballot_sync(0xffffffffu, is_tie);
                for (uint32_t ev = mm | tm; ev && g_hi < 0; ev &= ev - 1u) {
                  const int e = __ffs(ev) - 1;
                  if ((tm >> e) & 1u) {
                    ++ties;
                  } else {
                    const int gmark = (int)(__shfl_sync(0xffffffffu, w, e) & kMarkerMask);
                    if (ties >= need_t) {
                      g_hi = gmark;          // the batch that ends here holds the tie_need-th tie
                    } else {
                      g_lo = gmark;
                      ties_at_mark = ties;
                    }
                  }
                }
              }
              done += n_here;
              blk = __ldcg(b);
            }
            if (lane == rr && g_hi >= 0) {
              tie_pos_lo = g_lo << 3;
              tie_pos_hi = g_hi >= (int)kMarkerMask ? 0x7fffffff : g_hi << 3;
              tie_run = ties_at_mark;
            }
          }
          __syncwarp();
        }
      } else {   // kPassEmit: every resolved row appends its members in position order
        const bool em = row_ok && phase == kPhDone && n_keys > 0;
        int32_t* dst = sel_idx + ((int64_t)(r0 + (row_ok ? po : 0)) * d.n_ret + rh_head) * sel_stride;
        int run = 0;
        auto proc_e = [&](const uint32_t(&r)[16], const int n0) {
          const int valid = em ? pos - n0 + 1 : 0;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint32_t k = okey(finish_score(__uint_as_float(r[j]), scale));
            if (j < valid && (k > thr_key || (k == thr_key && n0 + j <= tie_last))) {
              if (run < sel_stride) dst[run] = n0 + j;
              ++run;
            }
          }
        };
#pragma unroll 1
        for (int it = t_lo; it < t_hi; ++it) {
          RTP_SEL_TILE_BEGIN
          (void)interior;
#define RTP_P(r_, n0_) proc_e(r_, n0_)
          RTP_SEL_GROUPS(RTP_P)
#undef RTP_P
          RTP_SEL_TILE_END
        }
        if (em && run > sel_stride) set_status(status, RTP_ERR_CAPACITY);
      }
#undef RTP_SEL_GROUPS
      if (kind != kPassEmit && phase != kPhDone) atomicOr(const_cast<int*>(&pass_flags[(pass + 1) & 1]), 1 << phase);
      if (kind != kPassEmit && phase == kPhTie) {
        atomicMin(&pass_rng[2 * ((pass + 1) & 1)], tie_pos_lo >> kPageShift);
        atomicMax(&pass_rng[2 * ((pass + 1) & 1) + 1], (int)min((unsigned)n_tiles, (((unsigned)tie_pos_hi - 1u) >> kPageShift) + 1u));
      }
    }
    sub_sync();
    if (tid == 0) {
      pass_flags[pass & 1] = 0;
      pass_rng[2 * (pass & 1)] = 0x7fffffff;
      pass_rng[2 * (pass & 1) + 1] = 0;
    }
    sub_sync();
  }

  // ---- results ----
  if (row_ok) {
    const int64_t o = (int64_t)(r0 + po) * d.n_ret + rh_head;
    if (phase != kPhDone) {
      set_status(status, RTP_ERR_TIMEOUT);
    }
    sel_count[o] = n_keys == 0 ? 0 : count;
    if (sel_mass) sel_mass[o] = sel_m;
    if (sel_thresh) sel_thresh[o] = thr_key == 0u ? -INFINITY : okey_to_float(thr_key);
    if (sel_tie_last) sel_tie_last[o] = n_keys == 0 ? -1 : tie_last;
  }
  }   // units
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_cta), "r"(kSubs * kTmemColsS) : "memory");
  }
}

template <int G>
cudaError_t launch_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                         const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride, int32_t* sel_count,
                         float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* ws,
                         size_t ws_bytes, int sm_count, cudaStream_t st) {
  static PerDeviceOnce once;
  cudaError_t e = set_dyn_smem_once(select_chunk_kernel<G>, kSmemS, once, true);
  if (e != cudaSuccess) return e;
  if (ws_bytes < 256 + (size_t)kBlockWords * 4) return cudaErrorInvalidValue;
  e = cudaMemsetAsync(ws, 0, 256, st);   // the pool's block counter
  if (e != cudaSuccess) return e;
  const size_t n_blocks = std::min<size_t>((ws_bytes - 256) / ((size_t)kBlockWords * 4), 0x7fffffffu);
  CUtensorMap map_ik;
  e = make_rows_map(&map_ik, cv.ikey, (int64_t)cv.num_pages * cv.n_ih * kPage, kIndexDim, kIndexDim, kPage,
                    (int)CU_TENSOR_MAP_SWIZZLE_32B);
  if (e != cudaSuccess) return e;
  constexpr int BMP = kSRows / G;
  const int n_row_tiles = (int)((rows.R + BMP - 1) / BMP);
  const int n_units = n_row_tiles * d.n_ih;
  dim3 grid(std::max(1, std::min(sm_count, (n_units + kSubs - 1) / kSubs)));
  const int mp = kMaxPasses;
  select_chunk_kernel<G><<<grid, kSubs * kSThreads, kSmemS, st>>>(map_ik, cv, d, hm, qt, rows.seq_id, rows.q_start, (int)rows.R,
                                                          sel_idx, sel_stride, sel_count, sel_mass, sel_thresh,
                                                          sel_tie_last, status, reinterpret_cast<uint32_t*>(ws) + 64, (uint32_t)n_blocks,
                                                          reinterpret_cast<unsigned int*>(ws), n_row_tiles, mp);
  return cudaGetLastError();
}

}  // namespace

// rows of a CTA are [head slot][position]: the smallest supported slot count that fits the widest index head
static int slot_class(const Dims& d, const HeadMaps& hm) {
  int max_nh = 0;
  for (int j = 0; j < d.n_ih; ++j) max_nh = hm.ih_nheads[j] > max_nh ? hm.ih_nheads[j] : max_nh;
  return max_nh <= 1 ? 1 : max_nh <= 2 ? 2 : max_nh <= 4 ? 4 : max_nh <= 8 ? 8 : 0;
}

// Workspace: a 256-byte header (the pool's block counter) and the block pool, kRowPoolEntries words per (row, head
// slot) of every unit.
size_t select_chunk_workspace_bytes(const Dims& d, const HeadMaps& hm, int64_t R) {
  const int g = slot_class(d, hm);
  if (g == 0 || R <= 0) return 256;
  const int64_t n_row_tiles = (R + kSRows / g - 1) / (kSRows / g);
  return 256 + (size_t)n_row_tiles * d.n_ih * kSRows * kRowPoolEntries * sizeof(uint32_t);
}

cudaError_t launch_select_chunk(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride,
                                int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                int32_t* status, void* ws, size_t ws_bytes, int sm_count, cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  if ((int64_t)rows.q_start + rows.R > (int64_t)1 << 21) return cudaErrorNotSupported;   // 8-bit overflow counters of the bins
  switch (slot_class(d, hm)) {
    case 1: return launch_typed<1>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, ws_bytes, sm_count, st);
    case 2: return launch_typed<2>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, ws_bytes, sm_count, st);
    case 4: return launch_typed<4>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, ws_bytes, sm_count, st);
    case 8: return launch_typed<8>(cv, d, hm, rows, qt, sel_idx, sel_stride, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, ws_bytes, sm_count, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace rtp
