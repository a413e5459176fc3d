// S6 / S7 / S9 for a prefill chunk on the 5th-generation tensor cores (tcgen05 + TMEM): dense, sink+window
// and sparse (Eq. 5) modes.
//
// One CTA (384 threads, one per SM) owns 128 MMA rows = (128 / G) consecutive positions x the G query
// heads of one KV head and walks the key tiles of 128 keys (two cache pages):
//   warps 9-10 loaders (K / V): pages -> shared memory in the 128-byte-swizzled layout the MMA unit reads; TMA
//             (cp.async.bulk.tensor, one lane) for whole tiles, zero-filling cp.async for the last tile; two stages
//   warp 8    one elected lane issues tcgen05.mma S = Q K^T (128 x 128 x 128) into one of two TMEM buffers
//   warp 11   one elected lane issues O += P V (128 x 128 x 128) once a softmax group has written P
//   warps 0-7 two softmax groups (even tiles / odd tiles) of 128 threads, thread = row = TMEM lane: read S with
//             tcgen05.ld, mask, online softmax, write P (bf16) to shared memory; each group accumulates its own
//             O in TMEM (rescaled there only when its reference maximum has to be raised); merged at the end.
//             Sparse mode: while the S MMA of its tile is in flight, each softmax warp re-evaluates the membership
//             of its 32 rows x 128 keys in S_h(m) from the 16-dim indexer scores (warp MMAs on index keys read
//             straight from the cache, the same arithmetic as the selection kernels) against the rows'
//             (threshold, tie position) pairs, and masks S with the resulting bits.
// Hand-offs are mbarriers (tcgen05.commit on the MMA side).  Every wait is bounded: when a wait runs
// out, the CTA records RTP_ERR_TIMEOUT, stops waiting (all later waits return at once), still walks its
// loops to the end, frees its TMEM and exits.
#include "tc_common.cuh"

namespace rtp {

namespace {

constexpr int kBM = 128;
constexpr int kBNt = 128;                 // keys per tile
constexpr int kTcThreads = 384;           // warps 0-7 softmax, 8 S-MMA issuer, 9 K loader, 10 V loader, 11 PV-MMA issuer
constexpr int kMmaWarp = 8, kLoadWarp0 = 9;   // warp 11 issues the P V MMAs
constexpr int kBlk = 128 * 128;           // bytes of one [128 rows][64 elements] bf16 block (16 KB)
constexpr int kQOff = 0;                  // Q: 2 blocks (dims 0-63, 64-127)
constexpr int kKOff = 2 * kBlk;           // K: 2 stages x 2 blocks
constexpr int kVOff = kKOff + 4 * kBlk;   // V: 2 stages x 2 blocks
constexpr int kPOff = kVOff + 4 * kBlk;   // P: 2 groups x 2 blocks (keys 0-63, 64-127)
constexpr int kBarOff = kPOff + 4 * kBlk; // mbarriers + TMEM base + abort flag
constexpr int kXchOff = kBarOff + 256;    // float [2 groups][2][128 rows]: (m, l) exchange for the final merge
constexpr int kTcSmem = kXchOff + 2048;
constexpr int kStageRow = 528;            // bytes per row of the fp32 staging tile used by the final merge (512 + 16)
constexpr float kLog2eT = 1.4426950408889634f;
constexpr float kLn2T = 0.6931471805599453f;

enum Bar { kFullK0 = 0, kFullK1, kFullV0, kFullV1, kEmptyK0, kEmptyK1, kEmptyV0, kEmptyV1, kSFull0, kSFull1, kSEmpty0, kSEmpty1,
           kPFull0, kPFull1, kPEmpty0, kPEmpty1, kNumBars };

// Shared-memory matrix descriptor, 128-byte swizzle.  sbo = byte distance between 8-row groups; lbo = byte
// distance between 64-element atoms along the contiguous dimension (only used by MN-major operands).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;   // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128; b_mn = B operand is MN-major (V as stored).
__device__ __forceinline__ uint32_t instr_desc(bool b_mn) {
  uint32_t d = 0;
  d |= 1u << 4;                     // D format fp32
  d |= 1u << 7;                     // A format bf16
  d |= 1u << 10;                    // B format bf16
  d |= (b_mn ? 1u : 0u) << 16;      // B major
  d |= (uint32_t)(kBNt >> 3) << 17; // N / 8
  d |= (uint32_t)(kBM >> 4) << 24;  // M / 16
  return d;
}
__device__ __forceinline__ void cp16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
// byte offset of 16-byte chunk c (0..7) of row r inside a [rows][64 elements] swizzled block
__device__ __forceinline__ uint32_t sw128(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

template <int G, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1) attn_prefill_tc_kernel(
    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
    const CacheView cv, const Dims d, const HeadMaps hm, const __nv_bfloat16* __restrict__ q,
    const __nv_bfloat16* __restrict__ qt, const float* __restrict__ sel_thresh, const int32_t* __restrict__ sel_tie_last,
    const int seq_id, const int q_start, const int C, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
    int32_t* status, const int n_row_tiles, const uint32_t* __restrict__ blk_mask, const int64_t mask_words) {
  constexpr int BMP = kBM / G;
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t sbase = s_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kBarOff + kNumBars * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kBarOff + kNumBars * 8 + 8);
  auto bar = [&](int i) { return sbase + kBarOff + i * 8; };

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = n_row_tiles - 1 - blockIdx.x;
  const int kvh = (MODE == kPrefillSparse || MODE == kPrefillBlocks) ? hm.ih_kv[blockIdx.y] : hm.kv_list[blockIdx.y];
  const int r0 = tile * BMP, m0 = q_start + r0;
  const int rows_here = min(BMP, C - r0);
  const int m_last = m0 + rows_here - 1;

  // key tiles of 128 keys visited by this CTA
  const int kt_last = m_last / kBNt;
  int kt_first = 0, n_sink_tiles = 0;
  if (MODE == kPrefillLocal) {
    kt_first = max(0, m0 - d.window + 1) / kBNt;
    n_sink_tiles = min((d.n_sink + kBNt - 1) / kBNt, kt_first);
  }
  const int n_tiles = n_sink_tiles + (kt_last - kt_first + 1);
  auto tile_at = [&](int i) { return i < n_sink_tiles ? i : kt_first + (i - n_sink_tiles); };

  if (tid == 0) {
    mbar_init(bar(kFullK0), 1); mbar_init(bar(kFullK1), 1);
    mbar_init(bar(kFullV0), 1); mbar_init(bar(kFullV1), 1);
    mbar_init(bar(kEmptyK0), 1); mbar_init(bar(kEmptyK1), 1);
    mbar_init(bar(kEmptyV0), 1); mbar_init(bar(kEmptyV1), 1);
    mbar_init(bar(kSFull0), 1); mbar_init(bar(kSFull1), 1);
    mbar_init(bar(kSEmpty0), 128); mbar_init(bar(kSEmpty1), 128);
    mbar_init(bar(kPFull0), 128); mbar_init(bar(kPFull1), 128);
    mbar_init(bar(kPEmpty0), 1); mbar_init(bar(kPEmpty1), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {   // TMEM: 512 columns (S0, S1, O_tile; one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Q tile -> shared (rows = [head][position]), by the softmax warps
  if (warp < 8) {
    for (int i = tid; i < kBM * 16; i += 256) {
      const int row = i >> 4, ch = i & 15;
      const int hs = row / BMP, po = row % BMP;
      const bool ok = po < rows_here;
      const __nv_bfloat16* src = q + ((int64_t)(r0 + (ok ? po : 0)) * d.n_q + kvh * d.group + hs) * kHeadDim + ch * 8;
      cp16(sbase + kQOff + (ch >> 3) * kBlk + sw128(row, ch & 7), src, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_s[2] = {tmem, tmem + 128u};          // S of the even-tile / odd-tile group
  const uint32_t tmem_o[2] = {tmem + 256u, tmem + 384u};   // their output accumulators

  // Register budget per role: the loader / issuer warpgroup hands registers back, the two softmax warpgroups (128
  // scores per thread live at once) take them: 256 x 232 + 128 x 40 = 384 x 168.
  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
  if (warp == kLoadWarp0 || warp == kLoadWarp0 + 1) {
    // ================================ loaders (warp 9: K tiles, warp 10: V tiles) ================================
    // Tiles whose 128 keys all exist are fetched by TMA (four 8 KB boxes, completion in bytes on the stage's
    // barrier; the warp does not wait for them).  The tile that holds the last position may reach into cache
    // slots that were never written: it is copied with cp.async and zero-filled beyond the last position.
    // A K stage is free again as soon as its S MMA has completed, a V stage once its P V MMA has.
    const int which = warp - kLoadWarp0;            // 0: K, 1: V
    const int64_t bt_base = (int64_t)seq_id * cv.max_pages;
    const int last_page = m_last >> kPageShift;
    const int rsub = lane >> 3, ch = lane & 7;     // 4 rows x 8 chunks per warp instruction
    const int kslot = cv.kv_slot[kvh];              // the KV head's place inside a page of this pool
    const __nv_bfloat16* pages = which ? cv.v : cv.k;
    const CUtensorMap* map = which ? &map_v : &map_k;
    for (int it = 0; it < n_tiles; ++it) {
      const int stage = it & 1;
      if (it >= 2) mbar_wait(bar((which ? kEmptyV0 : kEmptyK0) + stage), ((it >> 1) - 1) & 1, abort_flag, status, d.wait_ns);
      const int kt = tile_at(it);
      const uint32_t dst0 = sbase + (which ? kVOff : kKOff) + stage * 2 * kBlk;
      const uint32_t fb = bar((which ? kFullV0 : kFullK0) + stage);
      if (kt * kBNt + kBNt - 1 <= m_last) {
        if (lane == 0 && !(d.wait_test && which == 0 && it == 0)) {
          mbar_expect_tx(fb, 2 * kBlk);
#pragma unroll
          for (int pg = 0; pg < 2; ++pg) {
            const int phys = safe_phys(cv, bt_base + page_entry(cv, kt * 2 + pg), status);
            const int y = (phys * cv.n_kv + kslot) * kPage;
            tma_load_2d(dst0 + pg * (kPage * 128), map, 0, y, fb);
            tma_load_2d(dst0 + kBlk + pg * (kPage * 128), map, 64, y, fb);
          }
        }
        __syncwarp();
        continue;
      }
#pragma unroll 1
      for (int pg = 0; pg < 2; ++pg) {
        const int page = kt * 2 + pg;
        const bool page_ok = page <= last_page;
        const int phys = page_ok ? safe_phys(cv, bt_base + page_entry(cv, page), status) : 0;
        const __nv_bfloat16* src0 = pages + ((int64_t)phys * cv.n_kv + kslot) * (kPage * kHeadDim);
        const int n_ok = page_ok ? m_last - page * kPage + 1 : 0;   // keys of the page any row may attend
#pragma unroll 4
        for (int r4 = 0; r4 < 16; ++r4) {
          const int row = r4 * 4 + rsub;            // key inside the page
          const int trow = pg * kPage + row;        // key inside the tile
          const bool ok = row < n_ok;
          const __nv_bfloat16* src = src0 + (ok ? row : 0) * kHeadDim + ch * 8;
          cp16(dst0 + sw128(trow, ch), src, ok);                 // dims 0..63
          cp16(dst0 + kBlk + sw128(trow, ch), src + 64, ok);     // dims 64..127
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && !(d.wait_test && which == 0 && it == 0)) mbar_arrive(fb);   // (the test hook drops one signal)
    }
  } else if (warp == kMmaWarp) {
    // ================================ S = Q K^T issuer ================================
    // Runs ahead of the softmax groups: S_it only needs K_it and the S buffer of its group (released as soon as the
    // group has copied the previous S of that buffer into registers).
    const uint32_t idesc_s = instr_desc(false);
    for (int it = 0; it < n_tiles; ++it) {
      const int stage = it & 1, buf = it & 1;
      mbar_wait(bar(kFullK0 + stage), (it >> 1) & 1, abort_flag, status, d.wait_ns);
      if (it >= 2) mbar_wait(bar(kSEmpty0 + buf), ((it >> 1) - 1) & 1, abort_flag, status, d.wait_ns);
      tc_fence_after();
      if (lane == 0) {
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t da = smem_desc(sbase + kQOff + kb * kBlk + ks * 32, 16, 1024);
            const uint64_t db = smem_desc(sbase + kKOff + (stage * 2 + kb) * kBlk + ks * 32, 16, 1024);
            tc_mma(tmem_s[buf], da, db, idesc_s, (kb | ks) ? 1u : 0u);
          }
        tc_commit(bar(kSFull0 + buf));
        tc_commit(bar(kEmptyK0 + stage));
      }
      __syncwarp();
    }
  } else {
    // ================================ O_g += P V issuer ================================
    // g = it & 1: the even and the odd tiles are two independent online-softmax streams with their own accumulators
    const uint32_t idesc_o = instr_desc(true);
    for (int it = 0; it < n_tiles; ++it) {
      const int stage = it & 1, grp = it & 1;
      mbar_wait(bar(kFullV0 + stage), (it >> 1) & 1, abort_flag, status, d.wait_ns);
      mbar_wait(bar(kPFull0 + grp), (it >> 1) & 1, abort_flag, status, d.wait_ns);
      tc_fence_after();
      if (lane == 0) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {   // 16 keys per step
          const uint64_t da = smem_desc(sbase + kPOff + (grp * 2 + (ks >> 2)) * kBlk + (ks & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(sbase + kVOff + stage * 2 * kBlk + ks * 2048, kBlk, 1024);
          tc_mma(tmem_o[grp], da, db, idesc_o, ((it >> 1) | ks) ? 1u : 0u);
        }
        tc_commit(bar(kPEmpty0 + grp));
        tc_commit(bar(kEmptyV0 + stage));
      }
      __syncwarp();
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
    // ================================ softmax (two groups of 128 threads, thread = row) ================================
    // Group g (warps 4g .. 4g+3) handles the tiles it = g, g+2, ...: its own S buffer, P buffer and output
    // accumulator in TMEM, its own running (m_ref, l).  The two groups are independent online-softmax streams
    // over disjoint key tiles, so one group's exponentials overlap the other group's MMAs; they are merged once
    // at the end.  Probabilities are exp2(s - m_ref) with a reference that is only raised (and O, l rescaled in
    // TMEM) when a tile's maximum exceeds it by more than 8 in log2 units; any reference gives the same result
    // after the final division by l.
    const int grp = tid >> 7, row = tid & 127;
    const int hs = row / BMP, po = row % BMP;
    const bool row_ok = po < rows_here;
    const int pos = m0 + po;
    const int qh = kvh * d.group + hs;
    const float sc2 = d.sm_scale * kLog2eT;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    float* xch = reinterpret_cast<float*>(smem + kXchOff);
    float m_ref = -INFINITY, l_run = 0.f;
    int n_mine = 0;
    // ---- sparse mode: membership rule of the rows ----
    // Membership is tested on the unscaled MMA output: raw > up means "score above the row's threshold",
    // raw >= lo "at or above it" (they differ only for keys tied with the threshold score); upn is the next
    // float above up, so that raw > up <=> raw >= upn.  The per-row values live in shared memory (the region the
    // final merge reuses) and are re-read for every tile, like the projected-query fragments (from global
    // memory): nothing of the rule stays in registers across the softmax of a tile.
    const int ih = (MODE == kPrefillSparse || MODE == kPrefillBlocks) ? blockIdx.y : 0;
    // block mode: the row's page bits (one word per 32 pages)
    const uint32_t* mrow = (MODE == kPrefillBlocks && row_ok) ? blk_mask + ((int64_t)(r0 + po) * d.n_ret + hm.ih_heads[ih][hs]) * mask_words : nullptr;
    const int gq = lane >> 2, cq = lane & 3;
    float* thr_lo = xch;                                      // [128 rows]
    float* thr_upn = xch + 256;
    int* thr_tie = reinterpret_cast<int*>(xch + 384);
    int warp_pos_min = 0;
    const __nv_bfloat16* qt_lane = qt;                        // projected query of row (warp's first row + g), this lane's dims
    int qt_step[4] = {0, 0, 0, 0};                            // element offset of rows k*8 + g from it (-1: row absent)
    if (MODE == kPrefillSparse) {
      const float kInfT = __int_as_float(0x7f800000);
      if (grp == 0) {
        float lo_me = kInfT, up_me = kInfT;
        int tie_me = -1;
        if (row_ok) {
          const int64_t rr = (int64_t)(r0 + po) * d.n_ret + hm.ih_heads[ih][hs];
          const uint32_t tk = okey(sel_thresh[rr]);
          float dummy;
          raw_preimage(d.score_scale, tk, tk, lo_me, dummy);
          raw_preimage(d.score_scale, 0u, tk, dummy, up_me);
          tie_me = sel_tie_last[rr];
        }
        thr_lo[row] = lo_me;
        thr_upn[row] = (up_me < kInfT) ? okey_to_float(okey(up_me) + 1u) : kInfT;
        thr_tie[row] = tie_me;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      warp_pos_min = 0x7fffffff;
      const int row_w = (warp & 3) * 32;
      const int64_t base_rr = (int64_t)(r0 + (row_w + gq) % BMP) * d.n_ret + hm.ih_heads[ih][(row_w + gq) / BMP];
      qt_lane = qt + base_rr * kIndexDim + qfrag_dim_offset(lane);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int rowk = row_w + k * 8 + gq;
        const int hsk = rowk / BMP, pok = rowk % BMP;
        if (pok < rows_here) {
          warp_pos_min = min(warp_pos_min, m0 + pok);
          qt_step[k] = (int)(((int64_t)(r0 + pok) * d.n_ret + hm.ih_heads[ih][hsk] - base_rr) * kIndexDim);
        } else {
          qt_step[k] = -1;
        }
      }
      warp_pos_min = -__reduce_max_sync(0xffffffffu, -warp_pos_min);
    }
    const int64_t bt_base_s = (int64_t)seq_id * cv.max_pages;
    const int last_page_s = m_last >> kPageShift;
    // Index keys of a tile: lane (g, c) reads its 8 bytes of key 8 nt + g for every 8-key group nt.
    uint32_t iqa[2][4] = {{0u, 0u, 0u, 0u}, {0u, 0u, 0u, 0u}};   // A fragments of rows 0-15 / 16-31 of the warp
    if (MODE == kPrefillSparse) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint2 v = make_uint2(0u, 0u);
        if (qt_step[k] >= 0) v = __ldg(reinterpret_cast<const uint2*>(qt_lane + qt_step[k]));
        iqa[k >> 1][k & 1] = v.x;        // a0 (row g) / a1 (row g + 8)
        iqa[k >> 1][2 + (k & 1)] = v.y;  // a2 / a3
      }
    }

    for (int it = grp; it < n_tiles; it += 2, ++n_mine) {
      const int n_base = tile_at(it) * kBNt;
      uint32_t my[4] = {0u, 0u, 0u, 0u};   // this thread's row: bit 31 - (2 nt + e) of my[c] set <=> key 8 nt + 2 c + e is NOT a member
      if (MODE == kPrefillSparse) {
        // Tiles that are causal for every row of the warp and do not contain a row's tie position need one
        // comparison per score: raw >= lo before the tie position, raw > up (= raw >= upn) after it.  The sign
        // bits of (raw - threshold) are shifted into one word per row: the j-th appended element (j = 2 nt + e)
        // ends at bit 31 - j, set = NOT a member.
        uint32_t mw[4] = {0u, 0u, 0u, 0u};   // rows k*8 + g, columns 2 c, 2 c + 1 of every 8-key group
        float thr[4];
        bool fast = n_base + kBNt - 1 <= warp_pos_min;
        const int row_w = (warp & 3) * 32;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int rowk = row_w + k * 8 + gq;
          const int tie = thr_tie[rowk];
          const bool before = n_base + kBNt - 1 <= tie, after = tie < n_base;
          thr[k] = before ? thr_lo[rowk] : thr_upn[rowk];
          fast = fast && (before || after);
        }
        fast = __all_sync(0xffffffffu, fast);
        const float zero[4] = {0.f, 0.f, 0.f, 0.f};
        uint2 kb[16];
#pragma unroll
        for (int pg = 0; pg < 2; ++pg) {
          const int phys = safe_phys(cv, bt_base_s + min(n_base / kPage + pg, last_page_s), status);
          const __nv_bfloat16* ik =
              cv.ikey + ((int64_t)phys * cv.n_ih + ih) * (kPage * kIndexDim) + gq * kIndexDim + qfrag_dim_offset(lane);
#pragma unroll
          for (int n8 = 0; n8 < 8; ++n8) kb[pg * 8 + n8] = __ldg(reinterpret_cast<const uint2*>(ik + n8 * 8 * kIndexDim));
        }
        if (fast) {
#pragma unroll
          for (int nt = 0; nt < 16; ++nt) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              float s4[4];
              mma_bf16_16816(s4, iqa[t][0], iqa[t][1], iqa[t][2], iqa[t][3], kb[nt].x, kb[nt].y, zero);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int k = 2 * t + (e >> 1);
                mw[k] = __funnelshift_l(__float_as_uint(s4[e] - thr[k]), mw[k], 1);
              }
            }
          }
        } else {
          // general rule (diagonal tiles; tiles that hold the tie position of a row with tied keys left out): key n of
          // the tile belongs to the row's set iff n <= position and raw >= (n <= tie position ? lo : upn).  Rare, so
          // the loop stays rolled (small code): the 8-key group's fragment is picked from the registers by a switch-free
          // select chain.
          float lo_k[4], upn_k[4];
          int tie_rel[4], pos_rel[4];   // relative to the lane's first column of the tile
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int rowk = row_w + k * 8 + gq;
            lo_k[k] = thr_lo[rowk];
            upn_k[k] = thr_upn[rowk];
            tie_rel[k] = thr_tie[rowk] - n_base - 2 * cq;
            pos_rel[k] = m0 + rowk % BMP - n_base - 2 * cq;
          }
#pragma unroll 1
          for (int nt = 0; nt < 16; ++nt) {
            uint2 b = kb[0];
#pragma unroll
            for (int x = 1; x < 16; ++x)
              if (nt == x) b = kb[x];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              float s4[4];
              mma_bf16_16816(s4, iqa[t][0], iqa[t][1], iqa[t][2], iqa[t][3], b.x, b.y, zero);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int k = 2 * t + (e >> 1);
                const int j = nt * 8 + (e & 1);
                const float th = (j <= tie_rel[k]) ? lo_k[k] : upn_k[k];
                const bool in = (j <= pos_rel[k]) && (s4[e] >= th);
                mw[k] = (mw[k] << 1) | (in ? 0u : 1u);
              }
            }
          }
        }
        // lane (g, c) -> thread = row: row k*8 + g collects its four words from the lanes of quad g
        const int kk = lane >> 3;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int src = 4 * (lane & 7) + c;
          const uint32_t v0 = __shfl_sync(0xffffffffu, mw[0], src), v1 = __shfl_sync(0xffffffffu, mw[1], src);
          const uint32_t v2 = __shfl_sync(0xffffffffu, mw[2], src), v3 = __shfl_sync(0xffffffffu, mw[3], src);
          my[c] = kk == 0 ? v0 : kk == 1 ? v1 : kk == 2 ? v2 : v3;
        }
      }
      uint32_t page_bits = 3u;   // block mode: bit 0 / 1 = the tile's first / second page is selected by the row
      if (MODE == kPrefillBlocks) {
        const int pg = 2 * (n_base / kBNt);
        page_bits = mrow ? (__ldg(mrow + (pg >> 5)) >> (pg & 31)) & 3u : 0u;
      }
      mbar_wait(bar(kSFull0 + grp), n_mine & 1, abort_flag, status, d.wait_ns);
      tc_fence_after();
      float s[kBNt];
      {
        uint32_t* r0p = reinterpret_cast<uint32_t*>(s);
        uint32_t* r1p = r0p + 64;
        RTP_TMEM_LD64(r0p, tmem_s[grp] + lane_addr);
        RTP_TMEM_LD64(r1p, tmem_s[grp] + lane_addr + 64);
        tc_wait_ld();
      }
      tc_fence_before();
      mbar_arrive(bar(kSEmpty0 + grp));          // S is in registers: the buffer may be overwritten
      if (MODE == kPrefillSparse) {
#pragma unroll
        for (int i = 0; i < kBNt; ++i)
          if ((my[(i & 7) >> 1] >> (31 - (2 * (i >> 3) + (i & 1)))) & 1u) s[i] = -INFINITY;
      }
      if (MODE == kPrefillBlocks) {
        if (!(page_bits & 1u)) {
#pragma unroll
          for (int i = 0; i < kPage; ++i) s[i] = -INFINITY;
        }
        if (!(page_bits & 2u)) {
#pragma unroll
          for (int i = kPage; i < kBNt; ++i) s[i] = -INFINITY;
        }
      }
      bool need_mask = n_base + kBNt - 1 > pos;
      if (MODE == kPrefillLocal) need_mask = need_mask || (n_base <= pos - d.window);
      if (MODE == kPrefillSparse) need_mask = false;
      if (need_mask) {
#pragma unroll
        for (int i = 0; i < kBNt; ++i) {
          const int n = n_base + i;
          bool ok = n <= pos;
          if (MODE == kPrefillLocal) ok = ok && (n < d.n_sink || n > pos - d.window);
          if (!ok) s[i] = -INFINITY;
        }
      }
      float tmax;
      {
        float t0 = s[0], t1 = s[1], t2 = s[2], t3 = s[3];   // four independent chains
#pragma unroll
        for (int i = 4; i < kBNt; i += 4) {
          t0 = fmaxf(t0, s[i]); t1 = fmaxf(t1, s[i + 1]); t2 = fmaxf(t2, s[i + 2]); t3 = fmaxf(t3, s[i + 3]);
        }
        tmax = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3)) * sc2;
      }
      // this group's previous P must have been consumed (and its O must be quiescent) before P / O are touched
      if (n_mine >= 1) mbar_wait(bar(kPEmpty0 + grp), (n_mine - 1) & 1, abort_flag, status, d.wait_ns);
      const bool raise = tmax > m_ref + 8.0f;     // also true for the first finite maximum (m_ref = -inf)
      if (n_mine >= 1 && __any_sync(0xffffffffu, raise)) {
        tc_fence_after();
        const float f = raise ? ((m_ref == -INFINITY) ? 0.f : fast_ex2(m_ref - tmax)) : 1.f;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          uint32_t r[32];
          RTP_TMEM_LD32(r, tmem_o[grp] + lane_addr + c4 * 32);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
          RTP_TMEM_ST32(tmem_o[grp] + lane_addr + c4 * 32, r);
        }
        tc_wait_st();
        l_run *= f;
      }
      if (raise) m_ref = tmax;
      const float mb = (m_ref == -INFINITY) ? 0.f : m_ref;
      float rs[4] = {0.f, 0.f, 0.f, 0.f};
      unsigned char* pbase = smem + kPOff + grp * 2 * kBlk;
#pragma unroll
      for (int c8 = 0; c8 < 16; ++c8) {          // 8 keys = one 16-byte chunk of the row
        uint32_t pk[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float p0 = fast_ex2(fmaf(s[c8 * 8 + 2 * x], sc2, -mb)), p1 = fast_ex2(fmaf(s[c8 * 8 + 2 * x + 1], sc2, -mb));
          rs[x] += p0 + p1;
          __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
          pk[x] = *reinterpret_cast<uint32_t*>(&v);
        }
        *reinterpret_cast<uint4*>(pbase + (c8 >> 3) * kBlk + sw128(row, c8 & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
      l_run += (rs[0] + rs[1]) + (rs[2] + rs[3]);
      tc_fence_before();
      fence_async_smem();
      mbar_arrive(bar(kPFull0 + grp));
    }
    // ---- merge of the two groups and epilogue ----
    if (n_mine >= 1) mbar_wait(bar(kPEmpty0 + grp), (n_mine - 1) & 1, abort_flag, status, d.wait_ns);   // this group's last P V is done
    tc_fence_after();
    if (MODE == kPrefillSparse) asm volatile("bar.sync 1, 256;" ::: "memory");   // the rows' rule (same memory) is no longer read
    xch[(grp * 2 + 0) * 128 + row] = m_ref;
    xch[(grp * 2 + 1) * 128 + row] = l_run;
    asm volatile("bar.sync 1, 256;" ::: "memory");       // every MMA of the CTA has completed: shared memory is free
    const float m_oth = xch[((grp ^ 1) * 2 + 0) * 128 + row], l_oth = xch[((grp ^ 1) * 2 + 1) * 128 + row];
    const float m_tot = fmaxf(m_ref, m_oth);
    const float w_me = (m_ref == -INFINITY) ? 0.f : fast_ex2(m_ref - m_tot);
    const float w_ot = (m_oth == -INFINITY) ? 0.f : fast_ex2(m_oth - m_tot);
    const float l_tot = l_run * w_me + l_oth * w_ot;
    const float sc_me = l_tot > 0.f ? w_me / l_tot : 0.f;
    float* stage_row = reinterpret_cast<float*>(smem + kKOff + row * kStageRow);   // fp32 [128 dims] of group 1, scaled
    if (grp == 1) {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t r[32];
        if (n_mine >= 1) {
          RTP_TMEM_LD32(r, tmem_o[1] + lane_addr + c4 * 32);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          *reinterpret_cast<float4*>(stage_row + c4 * 32 + i) =
              make_float4(__uint_as_float(r[i]) * sc_me, __uint_as_float(r[i + 1]) * sc_me, __uint_as_float(r[i + 2]) * sc_me,
                          __uint_as_float(r[i + 3]) * sc_me);
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (grp == 0) {
      __nv_bfloat16* dst = out + ((int64_t)(r0 + (row_ok ? po : 0)) * d.n_q + qh) * kHeadDim;
      // (a local call computes a retrieval head that sits in a local group but leaves its slot to the sparse call)
      const bool row_wr = row_ok && !(MODE == kPrefillLocal && hm.skips(qh));
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t r[32];
        if (n_mine >= 1) {
          RTP_TMEM_LD32(r, tmem_o[0] + lane_addr + c4 * 32);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
        if (row_wr) {
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            const float4 a = *reinterpret_cast<const float4*>(stage_row + c4 * 32 + c8 * 8);
            const float4 b = *reinterpret_cast<const float4*>(stage_row + c4 * 32 + c8 * 8 + 4);
            const float o0 = fmaf(__uint_as_float(r[c8 * 8 + 0]), sc_me, a.x), o1 = fmaf(__uint_as_float(r[c8 * 8 + 1]), sc_me, a.y);
            const float o2 = fmaf(__uint_as_float(r[c8 * 8 + 2]), sc_me, a.z), o3 = fmaf(__uint_as_float(r[c8 * 8 + 3]), sc_me, a.w);
            const float o4 = fmaf(__uint_as_float(r[c8 * 8 + 4]), sc_me, b.x), o5 = fmaf(__uint_as_float(r[c8 * 8 + 5]), sc_me, b.y);
            const float o6 = fmaf(__uint_as_float(r[c8 * 8 + 6]), sc_me, b.z), o7 = fmaf(__uint_as_float(r[c8 * 8 + 7]), sc_me, b.w);
            __nv_bfloat162 v0 = __floats2bfloat162_rn(o0, o1), v1 = __floats2bfloat162_rn(o2, o3);
            __nv_bfloat162 v2 = __floats2bfloat162_rn(o4, o5), v3 = __floats2bfloat162_rn(o6, o7);
            *reinterpret_cast<uint4*>(dst + c4 * 32 + c8 * 8) =
                make_uint4(*reinterpret_cast<uint32_t*>(&v0), *reinterpret_cast<uint32_t*>(&v1), *reinterpret_cast<uint32_t*>(&v2),
                           *reinterpret_cast<uint32_t*>(&v3));
          }
        }
      }
      if (row_wr && lse) lse[(int64_t)(r0 + po) * d.n_q + qh] = l_tot > 0.f ? (m_tot + log2f(l_tot)) * kLn2T : -INFINITY;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// Tensor map over a paged cache viewed as [num_pages * n_kv * 64 rows][128 dims] bf16; box = 64 rows x 64 dims,
// 128-byte swizzle (the layout the MMA descriptors expect).
cudaError_t make_page_map(CUtensorMap* map, const void* base, int64_t rows) {
  return make_rows_map(map, base, rows, kHeadDim, 64, kPage, (int)CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int G, int MODE>
cudaError_t launch_tc_typed(const CacheView& cv, const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q,
                            const __nv_bfloat16* qt, const float* sel_thresh, const int32_t* sel_tie_last,
                            int32_t seq_id, int32_t q_start, int64_t C, __nv_bfloat16* out, float* lse,
                            int32_t* status, int n_units, cudaStream_t st, const uint32_t* blk_mask = nullptr,
                            int64_t mask_words = 0) {
  static PerDeviceOnce once;
  if (cudaError_t e0 = set_dyn_smem_once(attn_prefill_tc_kernel<G, MODE>, kTcSmem, once)) return e0;
  CUtensorMap map_k, map_v;
  const int64_t rows = (int64_t)cv.num_pages * cv.n_kv * kPage;
  cudaError_t e = make_page_map(&map_k, cv.k, rows);
  if (e != cudaSuccess) return e;
  e = make_page_map(&map_v, cv.v, rows);
  if (e != cudaSuccess) return e;
  constexpr int BMP = kBM / G;
  const int n_row_tiles = (int)((C + BMP - 1) / BMP);
  dim3 grid(n_row_tiles, n_units);
  attn_prefill_tc_kernel<G, MODE><<<grid, kTcThreads, kTcSmem, st>>>(map_k, map_v, cv, d, hm, q, qt, sel_thresh, sel_tie_last,
                                                                     seq_id, q_start, (int)C, out, lse, status, n_row_tiles, blk_mask,
                                                                     mask_words);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t launch_tc_mode(const CacheView& cv, const Dims& d, const HeadMaps& hm, const __nv_bfloat16* q,
                           const __nv_bfloat16* qt, const float* sel_thresh, const int32_t* sel_tie_last,
                           int32_t seq_id, int32_t q_start, int64_t C, __nv_bfloat16* out, float* lse, int32_t* status,
                           int n_units, cudaStream_t st, const uint32_t* blk_mask = nullptr, int64_t mask_words = 0) {
  switch (d.group) {
    case 1: return launch_tc_typed<1, MODE>(cv, d, hm, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, n_units, st, blk_mask, mask_words);
    case 2: return launch_tc_typed<2, MODE>(cv, d, hm, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, n_units, st, blk_mask, mask_words);
    case 4: return launch_tc_typed<4, MODE>(cv, d, hm, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, n_units, st, blk_mask, mask_words);
    case 8: return launch_tc_typed<8, MODE>(cv, d, hm, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, n_units, st, blk_mask, mask_words);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace

// Prefill attention on tcgen05: dense and sink+window over the KV heads of hm.kv_list, sparse (one CTA column per
// index head; the caller has checked that every index head serves the whole GQA group of its KV head).
cudaError_t launch_attn_prefill_tc(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                   const __nv_bfloat16* q, const __nv_bfloat16* qt, const float* sel_thresh,
                                   const int32_t* sel_tie_last, int32_t seq_id, int32_t q_start, int64_t C,
                                   __nv_bfloat16* out, float* lse, int32_t* status, cudaStream_t st,
                                   const uint32_t* blk_mask, int64_t mask_words) {
  if (C == 0) return cudaSuccess;
  if (mode == kPrefillBlocks)
    return d.n_ih == 0 ? cudaSuccess
                       : launch_tc_mode<kPrefillBlocks>(cv, d, hm, q, nullptr, nullptr, nullptr, seq_id, q_start, C, out, lse,
                                                        status, d.n_ih, st, blk_mask, mask_words);
  if (mode == kPrefillSparse)
    return d.n_ih == 0 ? cudaSuccess
                       : launch_tc_mode<kPrefillSparse>(cv, d, hm, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out,
                                                        lse, status, d.n_ih, st);
  if (hm.n_kv_list == 0) return cudaSuccess;
  if (mode == kPrefillLocal)
    return launch_tc_mode<kPrefillLocal>(cv, d, hm, q, nullptr, nullptr, nullptr, seq_id, q_start, C, out, lse, status,
                                         hm.n_kv_list, st);
  if (mode == kPrefillDense)
    return launch_tc_mode<kPrefillDense>(cv, d, hm, q, nullptr, nullptr, nullptr, seq_id, q_start, C, out, lse, status,
                                         hm.n_kv_list, st);
  return cudaErrorNotSupported;
}

// Prefill attention entry point of the library: every mode (dense, sink + window, sparse) runs on the tcgen05 kernel above.
cudaError_t launch_attn_prefill(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                const __nv_bfloat16* q, const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start,
                                int64_t C, const float* sel_thresh, const int32_t* sel_tie_last,
                                __nv_bfloat16* out, float* lse, int32_t* status, int sm_count, cudaStream_t st,
                                const uint32_t* blk_mask, int64_t mask_words) {
  (void)sm_count;
  if (C == 0) return cudaSuccess;
  if (mode == kPrefillSparse || mode == kPrefillBlocks) {
    // one CTA column per index head; every query head of its KV head must be a retrieval head on it
    for (int j = 0; j < d.n_ih; ++j)
      if (hm.ih_nheads[j] != d.group) return cudaErrorNotSupported;
    for (int i = 0; i < d.n_ret; ++i)
      if (hm.ret_q_head[i] != hm.ih_kv[hm.q2ih[i]] * d.group + hm.slot_in_ih[i]) return cudaErrorNotSupported;
    return launch_attn_prefill_tc(cv, d, hm, mode, q, qt, sel_thresh, sel_tie_last, seq_id, q_start, C, out, lse, status, st,
                                  blk_mask, mask_words);
  }
  if (hm.n_kv_list == 0) return cudaSuccess;
  return launch_attn_prefill_tc(cv, d, hm, mode, q, nullptr, nullptr, nullptr, seq_id, q_start, C, out, lse, status, st, nullptr, 0);
}

}  // namespace rtp
