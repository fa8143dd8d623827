// tcgen05/TMEM attention kernel (placeholder until the tensor-core path lands:
// reports every shape as unsupported, so the CUDA-core kernel is used).
#include "common.cuh"

namespace spiffy {

bool attention_tc_supported(const spiffy_attn_desc&) { return false; }
size_t attention_tc_workspace_bytes(const spiffy_attn_desc&) { return 0; }
spiffy_status launch_attention_tc(const spiffy_attn_desc&, const void*, const void*,
                                  const void*, const void*, const void*, void*,
                                  int32_t*, void*, cudaStream_t) {
  return SPIFFY_EUNSUPPORTED;
}

}  // namespace spiffy
