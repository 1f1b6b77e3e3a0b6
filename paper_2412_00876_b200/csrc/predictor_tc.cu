// Token predictor on the tensor cores (first line of Eq. 5 / Eq. 11 in per-token MLP form):
//   score[r] = w2 . GELU(W1 x_r + b1) + b2          bf16 inputs, fp32 accumulation
//
// A bf16 GEMM X[rows, d] * W1[p, d]^T on tcgen05 whose epilogue never materialises the hidden
// activations: each accumulator tile (128 rows x BN hidden units) is read from tensor memory one
// row per thread, biased, passed through the exact-erf GELU, multiplied by w2 and summed, all
// in fp32.  Persistent CTAs walk work items (row tile, unit tile) in an order that lets the CTAs
// that run side by side share one X tile through L2; a row tile's partial sums (one per unit
// tile) are added in tile order by the CTA that finishes last (a ticket, not a wait), so the
// logits are reproducible bit for bit.
//   warp 0 : TMA producer (X and W1 tiles, 128-byte swizzle, 4-stage ring)
//   warp 1 : tensor-memory allocation and the single MMA-issuing thread
//   warps 2-5 : epilogue, one TMEM lane quadrant each; two accumulators ping-pong so the epilogue
//               of one item overlaps the main loop of the next
// Every wait is bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kPtStages = 4;
constexpr int kPtBM = 128;
constexpr int kPtBK = 64;
constexpr int kPtMaxBN = 256;
constexpr int kPtThreads = 192;
constexpr int kPtATile = kPtBM * kPtBK * 2;          // 16 KB
constexpr int kPtBTile = kPtMaxBN * kPtBK * 2;       // 32 KB
constexpr int kPtStageBytes = kPtATile + kPtBTile;
constexpr size_t kPtSmem = (size_t)kPtStages * kPtStageBytes + 1024 /*align*/ + 256 /*barriers*/;

struct PredTcArgs {
  const float* b1; const float* w2; float b2;
  float* score; float* partial; int32_t* ticket; DeviceStatus* status;
  int32_t rows, rows_padded, k_blocks, bn, n_tiles, m_tiles, tmem_cols;
};

__global__ void __launch_bounds__(kPtThreads, 1)
predictor_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                    const PredTcArgs a) {
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kPtStages * kPtStageBytes);
  // bars: full[S] | empty[S] | acc_full[2] | acc_empty[2]
  uint64_t* full = bars;
  uint64_t* empty = bars + kPtStages;
  uint64_t* acc_full = bars + 2 * kPtStages;
  uint64_t* acc_empty = acc_full + 2;
  __shared__ uint32_t sh_tmem;
  __shared__ int sh_abort;
  __shared__ int sh_ticket;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh_abort;
  const int items = a.m_tiles * a.n_tiles;

  if (tid == 0) {
    sh_abort = 0;
    for (int s = 0; s < kPtStages; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_empty[i]), 4); }
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
  const uint32_t b_bytes = (uint32_t)a.bn * kPtBK * 2;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&map_x);
      tma_prefetch_desc(&map_w);
      int it = 0;
      for (int item = blockIdx.x; item < items && !*abort_flag; item += gridDim.x) {
        const int mt = item / a.n_tiles, nt = item - mt * a.n_tiles;
        for (int kb = 0; kb < a.k_blocks; ++kb, ++it) {
          const int s = it % kPtStages;
          if (!mbar_wait(smem_u32(&empty[s]), ((it / kPtStages) & 1) ^ 1, abort_flag)) break;
          const uint32_t fb = smem_u32(&full[s]);
          mbar_expect_tx(fb, kPtATile + b_bytes);
          char* st = smem + (size_t)s * kPtStageBytes;
          tma_load_2d(smem_u32(st), &map_x, kb * kPtBK, mt * kPtBM, fb);
          tma_load_2d(smem_u32(st + kPtATile), &map_w, kb * kPtBK, nt * a.bn, fb);
        }
      }
      if (*abort_flag) {
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        for (int j = max(0, it - kPtStages); j < it; ++j)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&full[j % kPtStages]), (j / kPtStages) & 1); ++i)
            __nanosleep(40);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(kPtBM, (uint32_t)a.bn);
      const uint64_t desc_a0 = smem_desc_sw128(smem_u32(smem));
      const uint64_t desc_b0 = smem_desc_sw128(smem_u32(smem) + kPtATile);
      int it = 0, j = 0;
      for (int item = blockIdx.x; item < items; item += gridDim.x, ++j) {
        const int buf = j & 1;
        mbar_wait(smem_u32(&acc_empty[buf]), ((j >> 1) & 1) ^ 1, abort_flag);
        tc_fence_after();
        const uint32_t d_tmem = tmem + (uint32_t)(buf * a.bn);
        for (int kb = 0; kb < a.k_blocks; ++kb, ++it) {
          const int s = it % kPtStages;
          mbar_wait(smem_u32(&full[s]), (it / kPtStages) & 1, abort_flag);
          tc_fence_after();
          // descriptors differ from the stage-0, k-0 ones only in the start-address field (16-byte units)
          const uint64_t da = desc_a0 + (uint64_t)((s * kPtStageBytes) >> 4);
          const uint64_t db = desc_b0 + (uint64_t)((s * kPtStageBytes) >> 4);
#pragma unroll
          for (int k = 0; k < kPtBK / 16; ++k)
            mma_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          mma_commit(smem_u32(&empty[s]));             // frees the stage when these MMAs have read it
        }
        mma_commit(smem_u32(&acc_full[buf]));          // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quad = warp & 3;                          // TMEM lanes 32*quad .. 32*quad+31
    const int et = (warp - 2) * 32 + lane;              // 0..127 among the epilogue threads
    int j = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, ++j) {
      const int mt = item / a.n_tiles, nt = item - mt * a.n_tiles;
      const int buf = j & 1;
      mbar_wait(smem_u32(&acc_full[buf]), (j >> 1) & 1, abort_flag);
      tc_fence_after();
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * a.bn);
      const float* b1 = a.b1 + (size_t)nt * a.bn;
      const float* w2 = a.w2 + (size_t)nt * a.bn;
      float sum = 0.f;
      for (int c = 0; c < a.bn; c += 32) {
        uint32_t r[32];
        tmem_ld32(t_row + c, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          sum = fmaf(__ldg(w2 + c + i), gelu_erf(__uint_as_float(r[i]) + __ldg(b1 + c + i)), sum);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
      const int row = mt * kPtBM + quad * 32 + lane;
      if (a.n_tiles == 1) {
        if (row < a.rows) a.score[row] = sum + a.b2;
        continue;
      }
      a.partial[(size_t)nt * a.rows_padded + row] = sum;
      __threadfence();
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (et == 0) sh_ticket = atomicAdd(&a.ticket[mt], 1);
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (sh_ticket == a.n_tiles - 1) {
        __threadfence();
        const int r2 = mt * kPtBM + et;
        float tot = 0.f;
        for (int t = 0; t < a.n_tiles; ++t) tot += __ldcg(a.partial + (size_t)t * a.rows_padded + r2);
        if (r2 < a.rows) a.score[r2] = tot + a.b2;
        if (et == 0) a.ticket[mt] = 0;
      }
    }
    if (*abort_flag && et == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
  }
}

bool predictor_tc_supported(const dl_ctx* ctx) {
  const dl_model_desc& d = ctx->desc;
  bool tile_ok = false;
  for (int cand : {256, 128, 64, 32})
    if (d.pred_hidden % cand == 0 && d.pred_hidden / cand <= kPredMaxSplit) tile_ok = true;
  return d.dtype == DL_BF16 && ctx->tmap_encode != nullptr && d.hidden % kPtBK == 0 && tile_ok &&
         (size_t)ctx->smem_optin >= kPtSmem;
}

cudaError_t launch_predictor_tc(dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows, float* score,
                                cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  const int m_tiles = (rows + kPtBM - 1) / kPtBM;
  // unit-tile width: the widest that still gives every SM an item, at most kPredMaxSplit tiles
  int bn = 0;
  for (int cand : {256, 128, 64, 32}) {
    if (d.pred_hidden % cand) continue;
    const int nt = d.pred_hidden / cand;
    if (nt > kPredMaxSplit) break;
    bn = cand;
    if (m_tiles * nt >= ctx->sm_count) break;
  }
  if (bn == 0) return cudaErrorInvalidValue;
  PredTcArgs a;
  a.b1 = p->b1; a.w2 = p->w2; a.b2 = p->b2; a.score = score;
  a.partial = ctx->ws.pred_partial; a.ticket = ctx->ws.pred_ticket; a.status = ctx->ws.status;
  a.rows = rows; a.rows_padded = ctx->ws.pred_rows_padded; a.k_blocks = d.hidden / kPtBK; a.bn = bn;
  a.n_tiles = d.pred_hidden / bn; a.m_tiles = m_tiles;
  int cols = 32;
  while (cols < 2 * bn) cols <<= 1;
  a.tmem_cols = cols;
  if (m_tiles * kPtBM > a.rows_padded) return cudaErrorInvalidValue;

  CUtensorMap mx, mw;
  const uint64_t dx[2] = {(uint64_t)d.hidden, (uint64_t)rows};
  const uint64_t dw[2] = {(uint64_t)d.hidden, (uint64_t)d.pred_hidden};
  const uint64_t st[1] = {(uint64_t)d.hidden * 2};
  const uint32_t bx[2] = {kPtBK, kPtBM};
  const uint32_t bw[2] = {kPtBK, (uint32_t)bn};
  if (!encode_bf16_map(ctx->tmap_encode, &mx, x, 2, dx, st, bx) ||
      !encode_bf16_map(ctx->tmap_encode, &mw, p->w1, 2, dw, st, bw))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(predictor_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPtSmem);
  if (e != cudaSuccess) return e;
  const int grid = min(ctx->sm_count, m_tiles * a.n_tiles);
  predictor_tc_kernel<<<grid, kPtThreads, kPtSmem, s>>>(mx, mw, a);
  return cudaGetLastError();
}

}  // namespace dl
