// Token predictor on CUDA cores (first line of Eq. 5 / Eq. 11 in per-token MLP form):
//   score[r] = w2 . GELU(W1 x_r + b1) + b2
// A shared-memory tiled fp32 GEMM whose epilogue applies bias, exact-erf GELU and the second
// layer, so the hidden activations never leave registers.  One CTA owns 32 rows and walks all
// hidden columns, which keeps the sum over columns in one fixed order.  This is the path for
// fp32 models and the fallback for bf16; the tensor-core kernel is in predictor_tc.cu.
#include "common.cuh"

namespace dl {

constexpr int PBM = 32, PBN = 64, PBK = 32, PTHREADS = 256;

template <typename T>
__global__ void __launch_bounds__(PTHREADS)
predictor_simt_kernel(const T* __restrict__ x, const T* __restrict__ w1, const float* __restrict__ b1,
                      const float* __restrict__ w2, float b2, int32_t rows, int32_t hidden,
                      int32_t pred_hidden, float* __restrict__ score) {
  __shared__ float As[PBK][PBM + 1];
  __shared__ float Bs[PBK][PBN + 1];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;          // 16 x 16 threads; thread tile 2 rows x 4 cols
  const int row0 = blockIdx.x * PBM;
  float rowsum[2] = {0.f, 0.f};

  for (int n0 = 0; n0 < pred_hidden; n0 += PBN) {
    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < hidden; k0 += PBK) {
      // A tile: 32 rows x 32 k  (1024 elements, 4 per thread)
      for (int e = tid; e < PBM * PBK; e += PTHREADS) {
        int r = e / PBK, kk = e - r * PBK;
        int gr = row0 + r, gk = k0 + kk;
        As[kk][r] = (gr < rows && gk < hidden) ? to_f32<T>(x[(size_t)gr * hidden + gk]) : 0.f;
      }
      // B tile: 64 hidden units x 32 k
      for (int e = tid; e < PBN * PBK; e += PTHREADS) {
        int n = e / PBK, kk = e - n * PBK;
        int gn = n0 + n, gk = k0 + kk;
        Bs[kk][n] = (gn < pred_hidden && gk < hidden) ? to_f32<T>(w1[(size_t)gn * hidden + gk]) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < PBK; ++kk) {
        float av[2] = {As[kk][ty * 2], As[kk][ty * 2 + 1]};
        float bv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      }
      __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn < pred_hidden) {
        float bb = b1[gn], ww = w2[gn];
#pragma unroll
        for (int i = 0; i < 2; ++i) rowsum[i] = fmaf(ww, gelu_erf(acc[i][j] + bb), rowsum[i]);
      }
    }
  }
  // the 16 threads that share a row are 16 consecutive lanes
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float v = rowsum[i];
    v += __shfl_xor_sync(0xffffffffu, v, 8);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    int gr = row0 + ty * 2 + i;
    if (tx == 0 && gr < rows) score[gr] = v + b2;
  }
}

cudaError_t launch_predictor_simt(const dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows,
                                  float* score, cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  dim3 grid((rows + PBM - 1) / PBM);
  if (d.dtype == DL_BF16)
    predictor_simt_kernel<__nv_bfloat16><<<grid, PTHREADS, 0, s>>>(
        (const __nv_bfloat16*)x, (const __nv_bfloat16*)p->w1, p->b1, p->w2, p->b2, rows, d.hidden,
        d.pred_hidden, score);
  else
    predictor_simt_kernel<float><<<grid, PTHREADS, 0, s>>>((const float*)x, (const float*)p->w1, p->b1,
                                                           p->w2, p->b2, rows, d.hidden, d.pred_hidden, score);
  return cudaGetLastError();
}

}  // namespace dl
