// Self-test of the bounded waits: a wait that can never be satisfied must end on its own, leave
// DL_ERR_TIMEOUT in the status word and return, with the context still usable.  Nothing here is on
// the hot path; the kernel holds no copy in flight and no tensor memory, so there is nothing to drain.
#include "common.cuh"
#include "pipeline.cuh"

namespace dl {

__global__ void wait_timeout_kernel(int polls, DeviceStatus* st) {
  __shared__ uint64_t bar;
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;
  if (threadIdx.x == 0) {
    sh_abort = 0;
    mbar_init(smem_u32(&bar), 2);          // two arrivals expected ...
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_arrive(smem_u32(&bar));      // ... one is made: the phase never completes
  __syncthreads();
  // the production wait (pipeline.cuh) with a short bound: gives up, raises the abort flag, returns false
  const bool ok = mbar_wait(smem_u32(&bar), 0, abort_flag, polls);
  // a second waiter sees the raised flag and leaves at once, as the roles of a pipelined kernel do
  const bool ok2 = mbar_wait(smem_u32(&bar), 0, abort_flag, polls);
  if (threadIdx.x == 0 && !ok && !ok2 && *abort_flag) report_status(st, DL_ERR_TIMEOUT, 0x5e1f);
}

}  // namespace dl

extern "C" int32_t dl_selftest_wait_timeout(dl_ctx* ctx, int32_t polls, void* stream) {
  if (!ctx || polls < 1 || polls > (1 << 16)) return DL_ERR_INVALID_ARG;
  if (!ctx->ws.base) return DL_ERR_WORKSPACE;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != ctx->device) cudaSetDevice(ctx->device);
  dl::wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(polls, ctx->ws.status);
  cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) { ctx->last_cuda = e; return DL_ERR_CUDA; }
  return DL_OK;
}
