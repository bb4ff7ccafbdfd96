// Placeholder until the tcgen05 scoring kernel lands.
#include "tensor_kernels.cuh"

namespace quoka {
bool score_keys_tc_supported(const quoka_params*) { return false; }
quoka_status launch_score_keys_tc(const quoka_params*, const DevParams&, const void*, const void*, float*,
                                  cudaStream_t) {
  return QUOKA_ERR_UNSUPPORTED;
}
}  // namespace quoka
