// Block-wise top-p selection for a prefill chunk (Section 3.4): the keys of a row are taken in blocks of one cache
// page (64 tokens), every block is reduced to a log-sum-exp pair (m_b, l_b) of its indexer scores, and blocks are
// selected in order of decreasing m_b until their softmax mass reaches p.  The result is one bit per (row, head, page).
//
// Same packaging as the token-level kernel: one persistent CTA per SM (a kernel that uses tensor memory runs alone
// on its SM) with four independent pipelines ("subs") of 128 threads; a sub takes units of 128 rows = (128 / G)
// consecutive positions x the G heads of one index head, thread = row = TMEM lane.
//   scan     the unit's pages once: index keys by TMA, S = Q~ K~^T (128 x 64 x 16) by tcgen05.mma into one of two TMEM
//            buffers, the thread reads its row's 64 scores and reduces them online to (m_b, l_b), which it stores
//            ([page][row]: a warp's store is contiguous), and keeps the row's maximum M and normaliser Z;
//   levels   the thread walks its own stored pairs (64 times fewer than scores): a 64-bin mass histogram, private to
//            the thread, first over a fixed quarter-wide grid of m_b below M, then over six more key bits per level,
//            always on the interval in which the mass crosses p Z; as soon as that interval holds at most eight
//            blocks they are ordered exactly (m_b descending, block index ascending); an interval of one key value
//            with more blocks is cut in index order;
//   emit     the pairs once more: bit b = block b is at or above the cut.
// No thread depends on another after the scan, so the levels need no barriers.
#include <algorithm>

#include "tc_common.cuh"

namespace rtp {

namespace {

constexpr int kBRows = 128;                     // rows (TMEM lanes) per unit
constexpr int kBStages = 4;                     // key pages in flight
constexpr int kBStageBytes = kPage * kIndexDim * 2;
constexpr int kBThreads = 128;                  // threads of a sub
constexpr int kBSubs = 4;
constexpr int kBTmemCols = 128;                 // two 64-column score buffers per sub
constexpr int kBBins = 64;
constexpr int kPoolBinB = 62;                   // grid level: bin that pools everything below the window (even shift)
constexpr int kMaxShiftB = kPoolBinB * 8;       // windows deeper than this hold no representable mass
constexpr int kCandB = 8;                       // blocks ordered exactly at the end
constexpr int kMaxLevelsB = 24;
constexpr float kLog2eB = 1.4426950408889634f;
constexpr float kMagicB = 12582912.0f;          // 1.5 * 2^23
constexpr uint32_t kMagicBitsB = 0x4B400000u;

constexpr int kBHistOff = 0;                                     // f32 [64 bins][128 rows]
constexpr int kBStageOff = kBBins * kBRows * 4;                  // kBStages x 2 KB
constexpr int kBAOff = kBStageOff + kBStages * kBStageBytes;     // projected queries [128 rows][16] bf16
constexpr int kBBarOff = kBAOff + kBRows * kIndexDim * 2;
constexpr int kBSmemSub = (kBBarOff + 256 + 1023) & ~1023;
constexpr int kBSmem = kBSubs * kBSmemSub;
enum BarB { kBFullK = 0, kBSFull = kBStages, kBNumBars = kBStages + 2 };

__device__ __forceinline__ float lds_f(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts_f(uint32_t a, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory"); }
// The stored pairs of a row are streamed through a small ring in shared memory with 8-byte cp.async copies, so that
// many pages are in flight per thread without holding them in registers.
constexpr int kRingDepth = 12;   // pages in flight per warp: 12 x 256 bytes (the key stages and the query tile are idle)
__device__ __forceinline__ void cp_async8(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ float2 lds_f2(uint32_t a) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void tmem_wait16b(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}
// Grid bin of a block maximum: round(-4 m) as an integer (monotone non-increasing in m; |m| < 2^18).
__device__ __forceinline__ int grid_bin_b(float s) { return (int)(__float_as_uint(fmaf(s, -4.0f, kMagicB)) - kMagicBitsB); }
// Exact interval [klo, khi] of ordered keys whose grid bin is `a`.
__device__ void grid_bin_keys_b(int a, uint32_t& klo, uint32_t& khi) {
  const float mid = -0.25f * (float)a;
  const uint32_t lo = okey(mid - 0.5f), hi = okey(mid + 0.5f);   // safely outside the bin on both sides
  uint32_t x = lo, y = hi;
  if (grid_bin_b(okey_to_float(x)) <= a) y = x;
  while (x + 1 < y) {
    const uint32_t m = x + ((y - x) >> 1);
    if (grid_bin_b(okey_to_float(m)) <= a) y = m; else x = m;
  }
  klo = y;
  x = klo; y = hi;
  if (grid_bin_b(okey_to_float(y)) >= a) x = y;
  while (x + 1 < y) {
    const uint32_t m = x + ((y - x) >> 1);
    if (grid_bin_b(okey_to_float(m)) >= a) x = m; else y = m;
  }
  khi = x;
}

template <int G>
__global__ void __launch_bounds__(kBSubs * kBThreads, 1) select_blocks_kernel(
    const __grid_constant__ CUtensorMap map_ik, const CacheView cv, const Dims d, const HeadMaps hm,
    const __nv_bfloat16* __restrict__ qt, const int seq_id, const int q_start, const int C,
    float2* __restrict__ stats, const int64_t slot_pages, uint32_t* __restrict__ mask, const int64_t mask_words,
    int32_t* __restrict__ sel_count, float* __restrict__ sel_mass, float* __restrict__ sel_thresh,
    int32_t* __restrict__ sel_tie_last, int32_t* status, const int n_row_tiles) {
  constexpr int BMP = kBRows / G;
  extern __shared__ __align__(1024) unsigned char smem_all[];
  const int sub = threadIdx.x / kBThreads;
  const int tid = threadIdx.x - sub * kBThreads, lane = tid & 31, warp = tid >> 5;
  unsigned char* smem = smem_all + sub * kBSmemSub;
  const uint32_t sbase = s_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_all + kBBarOff + kBNumBars * 8);   // (sub 0's slot serves the CTA)
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kBBarOff + kBNumBars * 8 + 4);
  unsigned int* rel = reinterpret_cast<unsigned int*>(smem + kBBarOff + kBNumBars * 8 + 16);   // [2] release tickets
  auto bar = [&](int i) { return sbase + kBBarOff + i * 8; };
  auto sub_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(1 + sub), "r"(kBThreads) : "memory"); };
  const int seq_len = min(cv.seq_lens[seq_id], cv.max_pages * kPage);   // (never beyond the block table)
  const float scale = d.score_scale;
  const float c2 = scale * kLog2eB;   // unscaled MMA output -> log2 units
  const int n_units = n_row_tiles * d.n_ih;

  if (tid == 0) {
    for (int i = 0; i < kBStages; ++i) mbar_init(bar(kBFullK + i), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kBSFull + i), 1);
      rel[i] = 0u;
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(kBSubs * kBTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_cta = *tmem_slot;
  const uint32_t tmem = tmem_cta + (uint32_t)(sub * kBTmemCols);
  // a warp reaches the 32 TMEM lanes of its quarter (warp index within the CTA modulo 4)
  const int quarter = (int)(threadIdx.x >> 5) & 3;
  const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
  const int row = quarter * 32 + lane;
  const uint32_t hist_col = sbase + kBHistOff + (uint32_t)row * 4u;
  constexpr uint32_t kStep = kBRows * 4;
  // the sub's slot of the pair buffer: [page][row]
  float2* my_stats = stats + ((int64_t)(blockIdx.x * kBSubs + sub) * slot_pages) * kBRows + row;

  uint32_t gt = 0;   // key pages consumed so far by this sub
  for (int unit = blockIdx.x + (int)gridDim.x * sub; unit < n_units; unit += (int)gridDim.x * kBSubs) {
    const int tile = n_row_tiles - 1 - unit / d.n_ih;
    const int ih = unit % d.n_ih;
    const int nh = hm.ih_nheads[ih];
    const int r0 = tile * BMP;
    const int rows_here = min(BMP, C - r0);
    const int m0 = q_start + r0;
    const int m_last = min(m0 + rows_here - 1, seq_len - 1);
    const int n_tiles = m_last >= 0 ? (m_last >> kPageShift) + 1 : 0;
    const int min_pos = min(m0, seq_len - 1);
    sub_sync();   // the previous unit's scan is finished by every thread of the sub
    if (tid == 0 && m0 + rows_here - 1 >= seq_len) set_status(status, RTP_ERR_INVALID);

    const int hs = row / BMP, po = row % BMP;
    const bool row_ok = hs < nh && po < rows_here;
    const int rh_head = hs < nh ? hm.ih_heads[ih][hs] : 0;
    const int pos = min(m0 + po, seq_len - 1);
    const int n_keys = row_ok ? pos + 1 : 0;
    const int nb_row = (n_keys + kPage - 1) >> kPageShift;   // blocks the row sees
    {
      // projected queries of the unit's rows -> the A operand (rows of 32 bytes, SWIZZLE_32B)
      uint4 v0 = make_uint4(0u, 0u, 0u, 0u), v1 = v0;
      if (row_ok) {
        const uint4* src = reinterpret_cast<const uint4*>(qt + ((int64_t)(r0 + po) * d.n_ret + rh_head) * kIndexDim);
        v0 = __ldg(src);
        v1 = __ldg(src + 1);
      }
      const int sw = (row >> 2) & 1;
      *reinterpret_cast<uint4*>(smem + kBAOff + row * 32 + ((0 ^ sw) << 4)) = v0;
      *reinterpret_cast<uint4*>(smem + kBAOff + row * 32 + ((1 ^ sw) << 4)) = v1;
      fence_async_smem();
    }
    sub_sync();

    const int64_t bt_base = (int64_t)seq_id * cv.max_pages;
    auto issue_tma = [&](uint32_t g, int page) {
      const int stage = (int)(g % kBStages);
      const int phys = safe_phys(cv, bt_base + page, status);
      mbar_expect_tx(bar(kBFullK + stage), kBStageBytes);
      tma_load_2d(sbase + kBStageOff + stage * kBStageBytes, &map_ik, 0, (phys * cv.n_ih + ih) * kPage, bar(kBFullK + stage));
    };
    auto issue_mma = [&](uint32_t g) {
      const int stage = (int)(g % kBStages), b2 = (int)(g & 1u);
      mbar_wait(bar(kBFullK + stage), (g / kBStages) & 1u, abort_flag, status, d.wait_ns);
      tc_fence_after();
      tc_mma(tmem + (uint32_t)(b2 * kPage), smem_desc_sw(sbase + kBAOff, 16, 256, 6),
             smem_desc_sw(sbase + kBStageOff + stage * kBStageBytes, 16, 256, 6), instr_desc_mn(kBRows, kPage, false), 0u);
      tc_commit(bar(kBSFull + b2));
    };
    if (warp == 0 && lane == 0) {
      for (int j = 0; j < kBStages && j < n_tiles; ++j) issue_tma(gt + (uint32_t)j, j);
      for (int j = 0; j < 2 && j < n_tiles; ++j) issue_mma(gt + (uint32_t)j);
    }
    __syncwarp();

    // ================================ scan: (m_b, l_b) of every page, M and Z of the row ================================
    float Mr = -INFINITY, Zr = 0.f;   // row maximum (unscaled MMA output) and sum of exp relative to it
#pragma unroll 1
    for (int it = 0; it < n_tiles; ++it) {
      const int buf = (int)(gt & 1u);
      mbar_wait(bar(kBSFull + buf), (gt >> 1) & 1u, abort_flag, status, d.wait_ns);
      tc_fence_after();
      const int n_base = it * kPage;
      const bool interior = n_base + kPage - 1 <= min_pos;
      const uint32_t taddr = tmem + lane_addr + (uint32_t)(buf * kPage);
      float mp = -INFINITY, lp = 0.f;   // the page's pair, online over its four groups of sixteen scores
      auto group = [&](const uint32_t(&r)[16], const int n0) {
        float g0 = -INFINITY, g1 = -INFINITY;
        if (interior) {
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            g0 = fmaxf(g0, __uint_as_float(r[j]));
            g1 = fmaxf(g1, __uint_as_float(r[j + 1]));
          }
        } else {
          const int valid = pos - n0 + 1;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < valid) g0 = fmaxf(g0, __uint_as_float(r[j]));
        }
        const float mn = fmaxf(mp, fmaxf(g0, g1));
        if (mn == -INFINITY) return;   // nothing of the group is visible to the row
        const float off = -mn * c2;
        float a0 = lp * fast_ex2(fmaf(mp, c2, off)), a1 = 0.f;   // (mp = -inf: the factor is 0)
        if (interior) {
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            a0 += fast_ex2(fmaf(__uint_as_float(r[j]), c2, off));
            a1 += fast_ex2(fmaf(__uint_as_float(r[j + 1]), c2, off));
          }
        } else {
          const int valid = pos - n0 + 1;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < valid) a0 += fast_ex2(fmaf(__uint_as_float(r[j]), c2, off));
        }
        lp = a0 + a1;
        mp = mn;
      };
      {
        uint32_t ra[16], rb[16];
        RTP_TMEM_LD16(ra, taddr);
        tmem_wait16b(ra);
        RTP_TMEM_LD16(rb, taddr + 16u);
        group(ra, n_base);
        tmem_wait16b(rb);
        RTP_TMEM_LD16(ra, taddr + 32u);
        group(rb, n_base + 16);
        tmem_wait16b(ra);
        RTP_TMEM_LD16(rb, taddr + 48u);
        group(ra, n_base + 32);
        tmem_wait16b(rb);
        group(rb, n_base + 48);
      }
      // hand the buffer on: the last of the four warps to release it issues the MMA of the page two ahead and requests
      // the keys of the page kBStages ahead
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        __threadfence_block();
        if (atomicAdd(&rel[buf], 1u) == 3u) {
          rel[buf] = 0u;
          tc_fence_after();
          if (it + 2 < n_tiles) issue_mma(gt + 2u);
          if (it + kBStages < n_tiles) issue_tma(gt + (uint32_t)kBStages, it + kBStages);
        }
      }
      __syncwarp();
      ++gt;
      const bool seen = row_ok && mp > -INFINITY;
      my_stats[(int64_t)it * kBRows] = make_float2(seen ? finish_score(mp, scale) : -INFINITY, seen ? lp : 0.f);
      if (seen) {
        const float mn = fmaxf(Mr, mp);
        Zr = Zr * fast_ex2((Mr - mn) * c2) + lp * fast_ex2((mp - mn) * c2);
        Mr = mn;
      }
    }

    // ---- the row's stored pairs, page after page (rows of a warp see at most one page more or less than each other) ----
    const int nb_warp = __reduce_max_sync(0xffffffffu, nb_row);
    const uint32_t ring = sbase + kBStageOff + (uint32_t)(warp * kRingDepth * 256 + lane * 8);
    auto for_pairs = [&](auto&& fn) {
#pragma unroll 1
      for (int k = 0; k < kRingDepth; ++k) {
        if (k < nb_warp) cp_async8(ring + (uint32_t)(k * 256), my_stats + (int64_t)k * kBRows);
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
      int slot = 0;
#pragma unroll 1
      for (int b = 0; b < nb_warp; ++b) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kRingDepth - 1) : "memory");
        const float2 v = lds_f2(ring + (uint32_t)(slot * 256));
        if (b + kRingDepth < nb_warp) cp_async8(ring + (uint32_t)(slot * 256), my_stats + (int64_t)(b + kRingDepth) * kBRows);
        asm volatile("cp.async.commit_group;" ::: "memory");
        slot = slot + 1 == kRingDepth ? 0 : slot + 1;
        if (b < nb_row) fn(b, v);
      }
      asm volatile("cp.async.wait_all;" ::: "memory");
    };
    // ================================ levels: the cut in (m_b descending, block ascending) order ================================
    if (row_ok) {
      const int64_t o = (int64_t)(r0 + po) * d.n_ret + rh_head;
      uint32_t thr_key = 0u;      // blocks with a larger key are selected, equal keys up to block tie_idx
      int tie_idx = nb_row - 1;
      float sel_m = 1.0f;
      bool done = n_keys == 0 || d.top_p >= 1.0f || nb_row <= 1;
      const float M = finish_score(Mr, scale), Z = Zr;
      const float target = d.top_p * Z;
      // mass of block (m, l) relative to exp(M)
      auto mass_of = [&](const float2 v) { return v.y * fast_ex2((v.x - M) * kLog2eB); };
      bool grid_level = true;
      // (even anchor and even window shifts: a maximum exactly between two bins is then binned as grid_bin_b says)
      const int aI = grid_bin_b(M) & ~1;
      int w0 = 0, shift = 0;
      uint32_t lo_key = 0u, span = 0u;
      float mass_above = 0.f;
#pragma unroll 1
      for (int level = 0; level < kMaxLevelsB && !done; ++level) {
        for (int b = 0; b < kBBins; ++b) sts_f(hist_col + (uint32_t)b * kStep, 0.f);
        int cnt = 0;
        uint32_t ck[kCandB];
        int cb[kCandB];
        float cm[kCandB];
#pragma unroll
        for (int k = 0; k < kCandB; ++k) {
          ck[k] = 0u;
          cb[k] = 0;
          cm[k] = 0.f;
        }
        const float dd = kMagicB - (float)(aI + w0);
        const bool tie_scan = !grid_level && span == 1u;
        float acc = mass_above;   // tie scan: mass up to and including the current block of the cut's key
        bool tie_found = false;
        for_pairs([&](const int b, const float2 v) {
          const float ms = mass_of(v);
          if (grid_level) {
            float t = fmaf(v.x, -4.0f, dd);
            if (!(t < kMagicB)) {   // (t < magic: above the window, counted by an earlier window)
              t = fminf(t, kMagicB + (float)kPoolBinB);
              const uint32_t a = hist_col + (__float_as_uint(t) & 63u) * kStep;
              sts_f(a, lds_f(a) + ms);
            }
          } else {
            const uint32_t t = okey(v.x) - lo_key;
            if (t < span) {
              if (tie_scan) {
                if (!tie_found) {
                  acc += ms;
                  tie_idx = b;
                  if (acc >= target) tie_found = true;
                }
              } else {
                const uint32_t a = hist_col + (t >> shift) * kStep;
                sts_f(a, lds_f(a) + ms);
#pragma unroll
                for (int q = 0; q < kCandB; ++q)
                  if (cnt == q) {
                    ck[q] = okey(v.x);
                    cb[q] = b;
                    cm[q] = ms;
                  }
                ++cnt;
              }
            }
          }
        });
        if (tie_scan) {
          thr_key = lo_key;
          sel_m = acc / Z;
          done = true;
        } else if (!grid_level && cnt <= kCandB) {
          // exact order of the few blocks left: largest key first, equal keys by block index
          float run = mass_above;
          uint32_t used = 0u;
          for (int step = 0; step < cnt; ++step) {
            int best = -1, bb = 0;
            uint32_t bk = 0u;
            float bm = 0.f;
#pragma unroll
            for (int q = 0; q < kCandB; ++q)
              if (q < cnt && !((used >> q) & 1u) && (best < 0 || ck[q] > bk || (ck[q] == bk && cb[q] < bb))) {
                best = q;
                bk = ck[q];
                bb = cb[q];
                bm = cm[q];
              }
            run += bm;
            thr_key = bk;
            tie_idx = bb;
            used |= 1u << best;
            if (run >= target) break;
          }
          sel_m = run / Z;
          done = true;
        } else {
          // bins in order of decreasing m_b: grid bins count up from the top, key bins down from 63
          float run = mass_above, above_found = 0.f, above_last = 0.f;
          int found = -1, last = -1;
          for (int i = 0; i < kBBins; ++i) {
            const int b = grid_level ? i : kBBins - 1 - i;
            const float h = lds_f(hist_col + (uint32_t)b * kStep);
            if (h > 0.f) {
              last = b;
              above_last = run;
              if (found < 0 && run + h >= target) {
                found = b;
                above_found = run;
              }
            }
            run += h;
          }
          if (found < 0) {   // rounding left the target just out of reach: the lowest populated bin
            found = last;
            above_found = above_last;
          }
          if (found < 0) {   // nothing below the mass already counted: every block is taken
            thr_key = 0u;
            tie_idx = nb_row - 1;
            sel_m = 1.0f;
            done = true;
          } else if (grid_level && found == kPoolBinB) {
            mass_above = above_found;
            w0 += kPoolBinB;
            if (w0 > kMaxShiftB) {
              thr_key = 0u;
              tie_idx = nb_row - 1;
              sel_m = 1.0f;
              done = true;
            }
          } else {
            mass_above = above_found;
            if (grid_level) {
              uint32_t klo, khi;
              grid_bin_keys_b(aI + w0 + found, klo, khi);
              lo_key = klo;
              span = khi - klo + 1u;
              grid_level = false;
            } else {
              const uint32_t ofs = (uint32_t)found << shift;
              lo_key += ofs;
              span = min(1u << shift, span - ofs);
            }
            const int bits = span > 1u ? 32 - __clz(span - 1u) : 0;
            shift = max(0, bits - 6);
          }
        }
      }
      if (!done) set_status(status, RTP_ERR_UNSUPPORTED);   // (more levels than a key has bits: cannot happen)

      // ================================ emit: one bit per block ================================
      int count = 0;
      uint32_t* mrow = mask + o * mask_words;
      const bool all = d.top_p >= 1.0f || nb_row <= 1 || thr_key == 0u;
      uint32_t bits = 0u;
      for_pairs([&](const int b, const float2 v) {
        const uint32_t key = okey(v.x);
        const bool sel = all || key > thr_key || (key == thr_key && b <= tie_idx);
        count += (int)sel;
        bits |= (sel ? 1u : 0u) << (b & 31);
        if ((b & 31) == 31 || b == nb_row - 1) {
          mrow[b >> 5] = bits;
          bits = 0u;
        }
      });
      sel_count[o] = count;
      if (sel_mass) sel_mass[o] = n_keys == 0 ? 0.f : (all ? 1.0f : sel_m);
      if (sel_thresh) sel_thresh[o] = (all || n_keys == 0) ? -INFINITY : okey_to_float(thr_key);
      if (sel_tie_last) sel_tie_last[o] = n_keys == 0 ? -1 : (all ? nb_row - 1 : tie_idx);
    }
  }   // units
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_cta), "r"(kBSubs * kBTmemCols) : "memory");
  }
}

int slot_class_b(const Dims& d, const HeadMaps& hm) {
  int max_nh = 0;
  for (int j = 0; j < d.n_ih; ++j) max_nh = hm.ih_nheads[j] > max_nh ? hm.ih_nheads[j] : max_nh;
  return max_nh <= 1 ? 1 : max_nh <= 2 ? 2 : max_nh <= 4 ? 4 : max_nh <= 8 ? 8 : 0;
}

template <int G>
cudaError_t launch_typed_b(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                           const __nv_bfloat16* qt, uint32_t* mask, int64_t mask_words, int32_t* sel_count,
                           float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* ws,
                           size_t ws_bytes, int sm_count, cudaStream_t st) {
  static PerDeviceOnce once;
  cudaError_t e = set_dyn_smem_once(select_blocks_kernel<G>, kBSmem, once, true);
  if (e != cudaSuccess) return e;
  CUtensorMap map_ik;
  e = make_rows_map(&map_ik, cv.ikey, (int64_t)cv.num_pages * cv.n_ih * kPage, kIndexDim, kIndexDim, kPage,
                    (int)CU_TENSOR_MAP_SWIZZLE_32B);
  if (e != cudaSuccess) return e;
  constexpr int BMP = kBRows / G;
  const int n_row_tiles = (int)((rows.R + BMP - 1) / BMP);
  const int n_units = n_row_tiles * d.n_ih;
  const int grid = std::max(1, std::min(sm_count, (n_units + kBSubs - 1) / kBSubs));
  const int64_t slot_pages = ((int64_t)rows.q_start + rows.R + kPage - 1) / kPage;
  if ((size_t)grid * kBSubs * slot_pages * kBRows * sizeof(float2) > ws_bytes) return cudaErrorInvalidValue;
  select_blocks_kernel<G><<<grid, kBSubs * kBThreads, kBSmem, st>>>(
      map_ik, cv, d, hm, qt, rows.seq_id, rows.q_start, (int)rows.R, reinterpret_cast<float2*>(ws), slot_pages, mask,
      mask_words, sel_count, sel_mass, sel_thresh, sel_tie_last, status, n_row_tiles);
  return cudaGetLastError();
}

}  // namespace

// Workspace: the pair buffer, one slot of ceil(max_len / 64) pages x 128 rows x 8 bytes per pipeline of the grid.
size_t select_blocks_workspace_bytes(const Dims& d, const HeadMaps& hm, int64_t R, int64_t max_len, int sm_count) {
  const int g = slot_class_b(d, hm);
  if (g == 0 || R <= 0) return 256;
  const int64_t n_units = ((R + kBRows / g - 1) / (kBRows / g)) * d.n_ih;
  const int64_t grid = std::max<int64_t>(1, std::min<int64_t>(sm_count, (n_units + kBSubs - 1) / kBSubs));
  const int64_t slot_pages = (max_len + kPage - 1) / kPage;
  return (size_t)grid * kBSubs * slot_pages * kBRows * sizeof(float2);
}

cudaError_t launch_select_blocks(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                 const __nv_bfloat16* qt, uint32_t* mask, int64_t mask_words, int32_t* sel_count,
                                 float* sel_mass, float* sel_thresh, int32_t* sel_tie_last, int32_t* status, void* ws,
                                 size_t ws_bytes, int sm_count, cudaStream_t st) {
  if (rows.R == 0 || d.n_ret == 0) return cudaSuccess;
  if ((int64_t)rows.q_start + rows.R > (int64_t)1 << 24) return cudaErrorNotSupported;
#define RTP_LB(GG) \
  return launch_typed_b<GG>(cv, d, hm, rows, qt, mask, mask_words, sel_count, sel_mass, sel_thresh, sel_tie_last, status, ws, ws_bytes, sm_count, st)
  switch (slot_class_b(d, hm)) {
    case 1: RTP_LB(1);
    case 2: RTP_LB(2);
    case 4: RTP_LB(4);
    case 8: RTP_LB(8);
    default: return cudaErrorNotSupported;
  }
#undef RTP_LB
}

}  // namespace rtp
