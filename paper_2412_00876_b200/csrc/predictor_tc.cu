// Tensor-core predictor (tcgen05): placeholder until the kernel lands.
#include "common.cuh"
namespace dl {
bool predictor_tc_supported(const dl_ctx*) { return false; }
cudaError_t launch_predictor_tc(dl_ctx*, const dl_predictor*, const void*, int32_t, float*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace dl
