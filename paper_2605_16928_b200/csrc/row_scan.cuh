// The scan of a row's index keys shared by the decode-time selection kernels: how a (row, index head) unit is split
// over CTAs, how a page of index keys is loaded, and which of the MMA's scores a lane post-processes.
#pragma once

#include "rtp_device.cuh"

namespace rtp {
namespace rowscan {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

struct RowCtx {
  int64_t r;
  int ih, split, seq, n_keys, p_lo, p_hi, nh;
};

__device__ __forceinline__ RowCtx make_row_ctx(const CacheView& cv, const Dims& d, const HeadMaps& hm,
                                               const Rows& rows, int n_splits, int32_t* status) {
  RowCtx x;
  x.r = blockIdx.x / d.n_ih;
  x.ih = blockIdx.x % d.n_ih;
  x.split = blockIdx.y;
  x.nh = hm.ih_nheads[x.ih];
  x.seq = rows.row_seq(x.r);
  int n_keys = rows.row_pos(x.r) + 1;
  const int sl = (x.seq >= 0 && x.seq < cv.batch) ? min(cv.seq_lens[x.seq], cv.max_pages * kPage) : 0;   // (never beyond the block table)
  if (n_keys > sl) {
    if (threadIdx.x == 0) set_status(status, RTP_ERR_INVALID);
    n_keys = sl;
  }
  if (n_keys < 0) n_keys = 0;
  x.n_keys = n_keys;
  const int n_pages = (n_keys + kPage - 1) >> kPageShift;
  const int per = (n_pages + n_splits - 1) / n_splits;
  x.p_lo = x.split * per;
  x.p_hi = min(n_pages, x.p_lo + per);
  return x;
}

// One 64-key page of index keys: 2 KB, four 16-byte loads per lane (bf16), or 1 KB, four 8-byte loads (E4M3: the
// upper half of each uint4 stays unused).
template <bool F8>
__device__ __forceinline__ void load_page(const CacheView& cv, const RowCtx& x, int p, int lane, uint4 (&v)[4]) {
  if (F8) {
    const uint8_t* base = ikey_page_ptr8(cv, x.seq, p, x.ih);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint2 t = ld_stream_v2(base + (i * 32 + lane) * 8);
      v[i].x = t.x;
      v[i].y = t.y;
    }
  } else {
    const __nv_bfloat16* base = ikey_page_ptr(cv, x.seq, p, x.ih);
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = ld_stream_v4(base + (i * 32 + lane) * 8);
  }
}

// ---- which scores a lane post-processes ------------------------------------------------------------
// After score16() lane (g, c) holds keys 4c .. 4c+3 of the 16-key group for head slots g (s_lo) and g + 8 (s_hi).
// With at most four heads on the index head (NH4) the lanes g >= 4 would idle: they take over keys 4c+2, 4c+3 of
// the lane that holds the same slot (g - 4), so that every lane handles two scores of slot g & 3.  Otherwise a lane
// handles four scores of slot g (set A) and four of slot g + 8 (set B).
template <bool NH4>
struct LaneElems {
  static constexpr int kN = NH4 ? 2 : 8;
  float raw[kN];
  int koff[kN];   // key offset inside the 16-key group
};
template <bool NH4>
__device__ __forceinline__ LaneElems<NH4> lane_elems(const float (&s_lo)[4], const float (&s_hi)[4], int lane) {
  LaneElems<NH4> r;
  const int c = lane & 3;
  if (NH4) {
    const float t2 = __shfl_sync(0xffffffffu, s_lo[2], lane & 15), t3 = __shfl_sync(0xffffffffu, s_lo[3], lane & 15);
    const bool up = lane >= 16;
    r.raw[0] = up ? t2 : s_lo[0];
    r.raw[1] = up ? t3 : s_lo[1];
    r.koff[0] = 4 * c + (up ? 2 : 0);
    r.koff[1] = r.koff[0] + 1;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      r.raw[e] = s_lo[e];
      r.raw[4 + e] = s_hi[e];
      r.koff[e] = r.koff[4 + e] = 4 * c + e;
    }
  }
  return r;
}
// head slot of element e of this lane
template <bool NH4>
__device__ __forceinline__ int elem_slot(int lane, int e) {
  const int g = lane >> 2;
  return NH4 ? (g & 3) : (e < 4 ? g : g + 8);
}

}  // namespace rowscan
}  // namespace rtp
