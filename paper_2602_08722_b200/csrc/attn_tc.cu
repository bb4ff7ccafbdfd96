// Placeholder until the tcgen05 attention kernel lands: reports "not covered" so the scalar kernel runs.
#include "tensor_kernels.cuh"

namespace quoka {
bool attn_tc_supported(const quoka_params*) { return false; }
quoka_status launch_attn_tc(const quoka_params*, const DevParams&, const void*, const void*, const void*,
                            const int32_t*, const int32_t*, void*, float*, cudaStream_t) {
  return QUOKA_ERR_UNSUPPORTED;
}
}  // namespace quoka
