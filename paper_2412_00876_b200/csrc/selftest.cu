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

// One checked store one element past the end of a 64-word buffer: the checked build must skip it and record it.
__global__ void bounds_selftest_kernel(int32_t* buf, int32_t n, DeviceStatus* st) {
  const int idx = n;                                    // one past the end
  if (DL_IN_BOUNDS(st, KID_SELFTEST, idx, n)) buf[idx] = 0x0bad;
}

}  // namespace dl

extern "C" int32_t dl_build_is_checked(void) {
#ifdef DL_BOUNDS
  return 1;
#else
  return 0;
#endif
}

extern "C" int32_t dl_selftest_bounds(dl_ctx* ctx, void* stream) {
  if (!ctx) return DL_ERR_INVALID_ARG;
  if (!ctx->ws.base) return DL_ERR_WORKSPACE;
#ifndef DL_BOUNDS
  (void)stream;
  return DL_ERR_UNSUPPORTED;
#else
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != ctx->device) cudaSetDevice(ctx->device);
  // the plan arrays of the workspace (max_batch words each, at least 64 with the padding of the layout) stand in
  // for "a small buffer"; the kernel is given 64 words of plan_base and must not touch word 64
  dl::bounds_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(ctx->ws.plan_base, 64, ctx->ws.status);
  cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) { ctx->last_cuda = e; return DL_ERR_CUDA; }
  return DL_OK;
#endif
}

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
