// S6 / S7 / S9 for a prefill chunk: placeholder until the tiled kernel lands.
#include "rtp_device.cuh"

namespace rtp {

cudaError_t launch_attn_prefill(const CacheView& cv, const Dims& d, const HeadMaps& hm, int mode,
                                const __nv_bfloat16* q, const __nv_bfloat16* qt, int32_t seq_id, int32_t q_start,
                                int64_t C, const float* sel_thresh, const int32_t* sel_tie_last,
                                __nv_bfloat16* out, float* lse, int32_t* status, int sm_count, cudaStream_t st) {
  return cudaErrorNotSupported;
}

}  // namespace rtp
