// Prefill attention over the reduced set on CUDA cores (Eq. 1 applied to S^{P*}):
// row i of a sequence's compact context attends rows 0..i of the same context.
// One warp per query row, 8 rows per CTA; 32-key tiles of K (transposed) and V are staged in
// shared memory as fp32, scores are one key per lane, the softmax is kept online per row.
// This is the path for fp32 models and head_dim 64 and the fallback for bf16; the tensor-core
// kernel is in attn_prefill_tc.cu.
#include "common.cuh"

namespace dl {

constexpr int kPfWarps = 8;

template <typename T, int D>
__global__ void __launch_bounds__(kPfWarps * 32)
attn_prefill_simt_kernel(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                         const int32_t* __restrict__ cache_len, int32_t H, int32_t cap, int32_t n_max,
                         float scale_log2, T* __restrict__ out, DeviceStatus* st) {
  __shared__ float Kt[D][33];
  __shared__ float Vs[32][D];
  __shared__ float Qs[kPfWarps][D];
  const int b = blockIdx.z, h = blockIdx.y, i0 = blockIdx.x * kPfWarps;
  const int n = min(max(cache_len[b], 0), min(cap, n_max));
  if (i0 >= n) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = i0 + warp;
  const bool row_ok = i < n;
  const size_t base = ((size_t)b * H + h) * cap * D;

  for (int d = lane; d < D; d += 32) Qs[warp][d] = row_ok ? to_f32<T>(q[base + (size_t)i * D + d]) * scale_log2 : 0.f;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[D / 32];
#pragma unroll
  for (int c = 0; c < D / 32; ++c) acc[c] = 0.f;

  const int last = min(i0 + kPfWarps - 1, n - 1);      // last key any row of this CTA may see
  for (int j0 = 0; j0 <= last; j0 += 32) {
    __syncthreads();
    for (int e = threadIdx.x; e < 32 * D; e += kPfWarps * 32) {
      int j = e / D, d = e - j * D;
      bool ok = (j0 + j) <= last;
      float kv = ok ? to_f32<T>(kc[base + (size_t)(j0 + j) * D + d]) : 0.f;
      float vv = ok ? to_f32<T>(vc[base + (size_t)(j0 + j) * D + d]) : 0.f;
      Kt[d][j] = kv;
      Vs[j][d] = vv;
    }
    __syncthreads();
    if (!row_ok || j0 > i) continue;
    float s = 0.f;
#pragma unroll 8
    for (int d = 0; d < D; ++d) s = fmaf(Qs[warp][d], Kt[d][lane], s);
    if (j0 + lane > i) s = -INFINITY;
    float mx = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float m_new = fmaxf(m_run, mx);
    const float corr = exp2f(m_run - m_new);
    const float p = exp2f(s - m_new);
    float ps = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    l_run = l_run * corr + ps;
    m_run = m_new;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) acc[c] *= corr;
    for (int j = 0; j < 32; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
      for (int c = 0; c < D / 32; ++c) acc[c] = fmaf(pj, Vs[j][lane + 32 * c], acc[c]);
    }
  }
  if (row_ok && DL_IN_BOUNDS(st, KID_PREFILL_SIMT, (((size_t)b * n_max + i) * H + h) * D + D - 1,
                             (size_t)gridDim.z * n_max * H * D)) {
    const float inv = 1.f / l_run;
    T* o = out + (((size_t)b * n_max + i) * H + h) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) o[lane + 32 * c] = from_f32<T>(acc[c] * inv);
  }
}

cudaError_t launch_attn_prefill_simt(const dl_ctx* ctx, const void* q, const void* k_cache,
                                     const void* v_cache, const int32_t* cache_len, int32_t B,
                                     int32_t cap, int32_t n_max, float scale, void* out, cudaStream_t s) {
  if (B == 0 || n_max == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  dim3 grid((n_max + kPfWarps - 1) / kPfWarps, d.n_heads, B);
  const float sl = scale * 1.4426950408889634f;
#define DL_LAUNCH(T, DD)                                                                              \
  attn_prefill_simt_kernel<T, DD><<<grid, kPfWarps * 32, 0, s>>>((const T*)q, (const T*)k_cache,       \
                                                                 (const T*)v_cache, cache_len, d.n_heads, \
                                                                 cap, n_max, sl, (T*)out,                        \
                                                                 ctx->ws.base ? ctx->ws.status : nullptr)
  if (d.dtype == DL_BF16) {
    if (d.head_dim == 128) DL_LAUNCH(__nv_bfloat16, 128);
    else if (d.head_dim == 64) DL_LAUNCH(__nv_bfloat16, 64);
    else return cudaErrorInvalidValue;
  } else {
    if (d.head_dim == 128) DL_LAUNCH(float, 128);
    else if (d.head_dim == 64) DL_LAUNCH(float, 64);
    else return cudaErrorInvalidValue;
  }
#undef DL_LAUNCH
  return cudaGetLastError();
}

}  // namespace dl
