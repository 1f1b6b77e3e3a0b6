// Tensor-core prefill attention (tcgen05): placeholder until the kernel lands.
#include "common.cuh"
namespace dl {
bool attn_prefill_tc_supported(const dl_ctx*) { return false; }
cudaError_t launch_attn_prefill_tc(dl_ctx*, const void*, const void*, const void*, const int32_t*, int32_t,
                                   int32_t, int32_t, float, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace dl
