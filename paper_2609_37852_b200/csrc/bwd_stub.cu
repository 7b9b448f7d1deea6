// Placeholders until the backward kernels land.
#include "common.cuh"
namespace attnfp8 {
attn_status_t launch_bwd_delta(const AttnShape&, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t,
                               const float*, float*, int*, cudaStream_t) {
  return fail(ATTN_ERR_UNSUPPORTED, "bwd_delta: not built yet");
}
attn_status_t launch_stale_delta(const AttnShape&, const void*, const void*, float*, cudaStream_t) {
  return fail(ATTN_ERR_UNSUPPORTED, "stale delta: not built yet");
}
attn_status_t launch_bwd_dq(const AttnShape&, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t,
                            const float*, const float*, void*, float*, float*, int*, cudaStream_t) {
  return fail(ATTN_ERR_UNSUPPORTED, "bwd dQ: not built yet");
}
attn_status_t launch_bwd_dkdv(const AttnShape&, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t, attn_qtensor_t,
                              const float*, const float*, void*, void*, int*, cudaStream_t) {
  return fail(ATTN_ERR_UNSUPPORTED, "bwd dK/dV: not built yet");
}
}  // namespace attnfp8
