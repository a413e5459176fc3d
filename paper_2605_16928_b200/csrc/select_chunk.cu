// S2-S4 for a prefill chunk: placeholder until the chunk kernel lands.
#include "rtp_device.cuh"

namespace rtp {

size_t select_chunk_workspace_bytes(const Dims& d, int64_t R) { return 256; }

cudaError_t launch_select_chunk(const CacheView& cv, const Dims& d, const HeadMaps& hm, const Rows& rows,
                                const __nv_bfloat16* qt, int32_t* sel_idx, int64_t sel_stride,
                                int32_t* sel_count, float* sel_mass, float* sel_thresh, int32_t* sel_tie_last,
                                int32_t* status, void* ws, int sm_count, cudaStream_t st) {
  return cudaErrorNotSupported;
}

}  // namespace rtp
