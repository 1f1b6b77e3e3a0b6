// Dense layer on the tensor cores for the paper's predictors (App. "Details of Predictor Architecture"):
//   C[M, N] = act(A[M, K] W[N, K]^T + bias)        A, W bf16, fp32 accumulation
// with the epilogue forms the predictor chain needs: bf16 or fp32 output, exact-erf GELU or none, and
// accumulation into an fp32 output (the residual stream of a transformer block).
// Same machinery as predictor_tc.cu: TMA (128-byte swizzle) -> 4-stage ring -> tcgen05.mma 128 x BN x 16,
// two accumulators in tensor memory so that the epilogue of one tile runs under the main loop of the next,
// persistent CTAs over (row tile, column tile) items with the column tiles of one row tile side by side (they
// share the A tile through L2).
//   warp 0 : TMA producer      warp 1 : tensor-memory allocation + the MMA-issuing thread
//   warps 2-9 : epilogue, two warps per TMEM lane quadrant (32-column chunks in turn), one output row per thread
// Every wait is bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kGmStages = 4, kGmBM = 128, kGmBK = 64, kGmMaxBN = 256, kGmThreads = 320;
constexpr int kGmATile = kGmBM * kGmBK * 2, kGmBTile = kGmMaxBN * kGmBK * 2, kGmStageBytes = kGmATile + kGmBTile;
constexpr size_t kGmSmem = (size_t)kGmStages * kGmStageBytes + 1024 + 256;

struct GemmArgs {
  const float* bias;        // [N] or null
  void* out;                // [M][ldo] bf16 or fp32
  DeviceStatus* status;
  int32_t M, N, k_blocks, bn, n_tiles, m_tiles, tmem_cols, ldo;
  int32_t out_f32, gelu, accumulate;
};

__global__ void __launch_bounds__(kGmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const GemmArgs a) {
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kGmStages * kGmStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kGmStages;
  uint64_t* acc_full = bars + 2 * kGmStages;
  uint64_t* acc_empty = acc_full + 2;
  __shared__ uint32_t sh_tmem;
  __shared__ int sh_abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh_abort;
  const int items = a.m_tiles * a.n_tiles;

  if (tid == 0) {
    sh_abort = 0;
    for (int s = 0; s < kGmStages; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_empty[i]), 8); }
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sh_tmem), (uint32_t)a.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh_tmem;
  const uint32_t b_bytes = (uint32_t)a.bn * kGmBK * 2;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&map_a);
      tma_prefetch_desc(&map_w);
      int it = 0;
      for (int item = blockIdx.x; item < items && !*abort_flag; item += gridDim.x) {
        const int mt = item / a.n_tiles, nt = item - mt * a.n_tiles;
        for (int kb = 0; kb < a.k_blocks; ++kb, ++it) {
          const int s = it % kGmStages;
          if (!mbar_wait(smem_u32(&empty[s]), ((it / kGmStages) & 1) ^ 1, abort_flag)) break;
          const uint32_t fb = smem_u32(&full[s]);
          mbar_expect_tx(fb, kGmATile + b_bytes);
          char* st = smem + (size_t)s * kGmStageBytes;
          tma_load_2d(smem_u32(st), &map_a, kb * kGmBK, mt * kGmBM, fb);
          tma_load_2d(smem_u32(st + kGmATile), &map_w, kb * kGmBK, nt * a.bn, fb);
        }
      }
      if (*abort_flag) {
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        for (int j = max(0, it - kGmStages); j < it; ++j)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&full[j % kGmStages]), (j / kGmStages) & 1); ++i)
            __nanosleep(40);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(kGmBM, (uint32_t)a.bn);
      const uint64_t desc_a0 = smem_desc_sw128(smem_u32(smem));
      const uint64_t desc_b0 = smem_desc_sw128(smem_u32(smem) + kGmATile);
      int it = 0, j = 0;
      for (int item = blockIdx.x; item < items; item += gridDim.x, ++j) {
        const int buf = j & 1;
        mbar_wait(smem_u32(&acc_empty[buf]), ((j >> 1) & 1) ^ 1, abort_flag);
        tc_fence_after();
        const uint32_t d_tmem = tmem + (uint32_t)(buf * a.bn);
        for (int kb = 0; kb < a.k_blocks; ++kb, ++it) {
          const int s = it % kGmStages;
          mbar_wait(smem_u32(&full[s]), (it / kGmStages) & 1, abort_flag);
          tc_fence_after();
          const uint64_t da = desc_a0 + (uint64_t)((s * kGmStageBytes) >> 4);
          const uint64_t db = desc_b0 + (uint64_t)((s * kGmStageBytes) >> 4);
#pragma unroll
          for (int k = 0; k < kGmBK / 16; ++k) mma_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          mma_commit(smem_u32(&empty[s]));
        }
        mma_commit(smem_u32(&acc_full[buf]));
      }
    }
  } else {
    // a warp reads the TMEM lanes of quadrant warp % 4; the two warps of a quadrant take the 32-column chunks in turn
    const int quad = warp & 3, half = (warp - 2) >> 2;
    int j = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, ++j) {
      const int mt = item / a.n_tiles, nt = item - mt * a.n_tiles;
      const int buf = j & 1;
      mbar_wait(smem_u32(&acc_full[buf]), (j >> 1) & 1, abort_flag);
      tc_fence_after();
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * a.bn);
      const int row = mt * kGmBM + quad * 32 + lane;
      const int col0 = nt * a.bn;
      if (32 * half >= a.bn) {                      // a tile of one chunk: nothing for the second warp of the quadrant
        if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
        continue;
      }
      for (int c = 32 * half; c < a.bn; c += 64) {
        uint32_t r[32];
        tmem_ld32(t_row + c, r);
        tmem_ld_wait();
        if (c + 64 >= a.bn) {                       // this warp's share is in registers: the next tile may use it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
        }
        if (row >= a.M) continue;
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float y = __uint_as_float(r[i]) + (a.bias ? __ldg(a.bias + col0 + c + i) : 0.f);
          v[i] = a.gelu ? gelu_erf(y) : y;
        }
        if (a.out_f32) {
          float4* o = reinterpret_cast<float4*>(static_cast<float*>(a.out) + (size_t)row * a.ldo + col0 + c);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 w = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            if (a.accumulate) { const float4 p = o[i]; w.x += p.x; w.y += p.y; w.z += p.z; w.w += p.w; }
            o[i] = w;
          }
        } else {
          uint4* o = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(a.out) + (size_t)row * a.ldo + col0 + c);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 w;
            __nv_bfloat162 t0 = __floats2bfloat162_rn(v[8 * i], v[8 * i + 1]), t1 = __floats2bfloat162_rn(v[8 * i + 2], v[8 * i + 3]);
            __nv_bfloat162 t2 = __floats2bfloat162_rn(v[8 * i + 4], v[8 * i + 5]), t3 = __floats2bfloat162_rn(v[8 * i + 6], v[8 * i + 7]);
            w.x = *reinterpret_cast<uint32_t*>(&t0); w.y = *reinterpret_cast<uint32_t*>(&t1);
            w.z = *reinterpret_cast<uint32_t*>(&t2); w.w = *reinterpret_cast<uint32_t*>(&t3);
            o[i] = w;
          }
        }
      }
    }
    if (*abort_flag && warp == 2 && lane == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
  }
}

bool gemm_tc_supported(const dl_ctx* ctx) { return ctx->tmap_encode != nullptr && (size_t)ctx->smem_optin >= kGmSmem; }

// A [M][K] bf16 (K a multiple of 64), W [N][K] bf16 (N a multiple of 32), out [M][ldo]; all 16-byte aligned.
cudaError_t launch_gemm_tc(const dl_ctx* ctx, const void* A, const void* W, const float* bias, void* out, int M, int N,
                           int K, int ldo, bool out_f32, bool gelu, bool accumulate, cudaStream_t s) {
  if (M == 0 || N == 0) return cudaSuccess;
  if (K % kGmBK || N % 32 || !gemm_tc_supported(ctx)) return cudaErrorInvalidValue;
  const int m_tiles = (M + kGmBM - 1) / kGmBM;
  int bn = 0;
  for (int cand : {256, 128, 64, 32}) {
    if (N % cand) continue;
    bn = cand;
    if (m_tiles * (N / cand) >= ctx->sm_count) break;
  }
  GemmArgs a;
  a.bias = bias; a.out = out; a.status = ctx->ws.base ? ctx->ws.status : nullptr;
  a.M = M; a.N = N; a.k_blocks = K / kGmBK; a.bn = bn; a.n_tiles = N / bn; a.m_tiles = m_tiles; a.ldo = ldo;
  a.out_f32 = out_f32; a.gelu = gelu; a.accumulate = accumulate;
  int cols = 32;
  while (cols < 2 * bn) cols <<= 1;
  a.tmem_cols = cols;
  CUtensorMap ma, mw;
  const uint64_t da[2] = {(uint64_t)K, (uint64_t)M}, dw[2] = {(uint64_t)K, (uint64_t)N};
  const uint64_t st[1] = {(uint64_t)K * 2};
  const uint32_t ba[2] = {kGmBK, kGmBM}, bw[2] = {kGmBK, (uint32_t)bn};
  if (!encode_bf16_map(ctx->tmap_encode, &ma, A, 2, da, st, ba) || !encode_bf16_map(ctx->tmap_encode, &mw, W, 2, dw, st, bw))
    return cudaErrorInvalidValue;
  static int attr_set[64];
  if (!attr_set[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGmSmem);
    if (e != cudaSuccess) return e;
    attr_set[ctx->device & 63] = 1;
  }
  const int grid = std::min(ctx->sm_count, m_tiles * a.n_tiles);
  gemm_tc_kernel<<<grid, kGmThreads, kGmSmem, s>>>(ma, mw, a);
  return cudaGetLastError();
}

}  // namespace dl
