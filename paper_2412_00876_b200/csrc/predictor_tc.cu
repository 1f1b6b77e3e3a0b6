// Token predictor on the tensor cores (first line of Eq. 5 / Eq. 11 in per-token MLP form):
//   score[r] = w2 . GELU(W1 x_r + b1) + b2          bf16 inputs, fp32 accumulation
//
// A bf16 GEMM X[rows, d] * W1[p, d]^T on tcgen05 whose epilogue never materialises the hidden
// activations: each accumulator tile (128 rows x BN hidden units) is read from tensor memory one
// row per thread, biased, passed through the exact-erf GELU, multiplied by w2 and summed, all
// in fp32.  Persistent CTAs walk work items (row tile, unit tile) in an order that lets the CTAs
// that run side by side share one X tile through L2; a row tile's partial sums (one per unit
// tile) are added in tile order by the CTA that finishes last (a ticket, not a wait), so the
// logits are reproducible bit for bit.  With a single row tile (the decode shape: one row per sequence) the
// hidden dimension is also split over CTAs: each takes a range of it for its unit tile, leaves the raw fp32
// sums in scratch, and the last of a unit tile's CTAs to arrive adds the ranges in order before the GELU.
//   warp 0 : TMA producer (X and W1 tiles, 128-byte swizzle; a ring of 4 stages for prefill shapes, up to 32
//            short stages for the few rows of a decode step)
//   warp 1 : tensor-memory allocation and the single MMA-issuing thread
//   warps 2-5 : epilogue, one TMEM lane quadrant each; two accumulators ping-pong so the epilogue
//               of one item overlaps the main loop of the next
// Every wait is bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kPtMaxStages = 32;
constexpr int kPtBM = 128;
constexpr int kPtBK = 64;
constexpr int kPtMaxBN = 256;
constexpr int kPtThreads = 192;
constexpr int kPtATile = kPtBM * kPtBK * 2;          // 16 KB
constexpr int kPtBTile = kPtMaxBN * kPtBK * 2;       // 32 KB
constexpr int kPtStageBytes = kPtATile + kPtBTile;   // a stage of the widest form (128 rows, 256 units)
constexpr int kPtBarBytes = (2 * kPtMaxStages + 4) * 8;
// the ring, then room for the MMA's 128-row read past a short last stage, the barriers, the alignment slack
constexpr size_t kPtSmem = (size_t)4 * kPtStageBytes + kPtATile + kPtBarBytes + 1024;

struct PredTcArgs {
  const float* b1; const float* w2; float b2;
  float* score; float* partial; int32_t* ticket; DeviceStatus* status;
  int32_t rows, rows_padded, k_blocks, bn, n_tiles, m_tiles, tmem_cols;
  int32_t stages, stage_bytes, a_bytes;   // ring depth; bytes per stage; bytes of its X part
  int32_t kbs, a_tile, b_tile;            // 64-column blocks of the hidden dimension per stage; bytes of one X / one W1 block
  uint8_t* keep; float threshold;         // decode decision fused into the final sum (keep may be null)
  int32_t row_box;                        // rows of X fetched per stage (32, 64 or 128); below 128 only with one row tile
  int32_t k_split, kb_per;                // CTAs per unit tile along the hidden dimension; 64-column blocks each takes
  float* split; int32_t* split_ticket;    // [n_tiles][k_split][128][bn] raw sums; [n_tiles] arrivals, zero between launches
};

// score and, if asked for, the decision keep = score > threshold (strictly; a NaN score drops and is reported)
__device__ __forceinline__ void pt_emit(const PredTcArgs& a, int row, float score) {
  a.score[row] = score;
  if (a.keep != nullptr) {
    if (score != score) report_status(a.status, DL_WARN_NAN, row);
    a.keep[row] = score > a.threshold ? 1 : 0;
  }
}

__global__ void __launch_bounds__(kPtThreads, 1)
predictor_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                    const PredTcArgs a) {
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NS = a.stages;
  // The MMA always reads 128 rows of X from a stage; with a short row box (few rows: the decode shape) the rows
  // past the box are whatever follows in shared memory, and their results are never stored.
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)NS * a.stage_bytes + kPtATile);
  // bars: full[S] | empty[S] | acc_full[2] | acc_empty[2]
  uint64_t* full = bars;
  uint64_t* empty = bars + NS;
  uint64_t* acc_full = bars + 2 * NS;
  uint64_t* acc_empty = acc_full + 2;
  __shared__ uint32_t sh_tmem;
  __shared__ int sh_abort;
  __shared__ int sh_ticket;
  __shared__ float sh_red[4][kPtBM];      // sums of the threads that share a row, added in order by the row's first thread

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh_abort;
  const int items = a.m_tiles * a.n_tiles * a.k_split;

  if (tid == 0) {
    sh_abort = 0;
    for (int s = 0; s < NS; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1); }
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
  const uint32_t b_bytes = (uint32_t)(a.kbs * a.b_tile);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&map_x);
      tma_prefetch_desc(&map_w);
      int it = 0, s = 0, ph = 0;                 // stage and phase of fill `it`, kept by counting (NS is a run-time value)
      for (int item = blockIdx.x; item < items && !*abort_flag; item += gridDim.x) {
        const int tile = item / a.k_split, sp = item - tile * a.k_split;
        const int mt = tile / a.n_tiles, nt = tile - mt * a.n_tiles;
        const int kb_end = min(a.k_blocks, (sp + 1) * a.kb_per);
        for (int kb = sp * a.kb_per; kb < kb_end; kb += a.kbs, ++it) {
          if (!mbar_wait(smem_u32(&empty[s]), ph ^ 1, abort_flag)) break;
          const uint32_t fb = smem_u32(&full[s]);
          mbar_expect_tx(fb, (uint32_t)a.a_bytes + b_bytes);
          char* st = smem + (size_t)s * a.stage_bytes;
          // one copy each for the stage's kbs blocks of X and of W1: the maps see the hidden dimension as
          // (64 columns, row, block), so the blocks land one after the other as K-major tiles
          tma_load_3d(smem_u32(st), &map_x, 0, mt * kPtBM, kb, fb);
          tma_load_3d(smem_u32(st + a.a_bytes), &map_w, 0, nt * a.bn, kb, fb);
          if (++s == NS) { s = 0; ph ^= 1; }
        }
      }
      if (*abort_flag) {
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        for (int j = max(0, it - NS); j < it; ++j)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&full[j % NS]), (j / NS) & 1); ++i)
            __nanosleep(40);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(kPtBM, (uint32_t)a.bn);
      const uint64_t desc_a0 = smem_desc_sw128(smem_u32(smem));
      const uint64_t desc_b0 = smem_desc_sw128(smem_u32(smem) + (uint32_t)a.a_bytes);
      int s = 0, ph = 0, j = 0;
      for (int item = blockIdx.x; item < items; item += gridDim.x, ++j) {
        const int buf = j & 1;
        mbar_wait(smem_u32(&acc_empty[buf]), ((j >> 1) & 1) ^ 1, abort_flag);
        tc_fence_after();
        const uint32_t d_tmem = tmem + (uint32_t)(buf * a.bn);
        const int sp = item % a.k_split;
        const int kb0 = sp * a.kb_per, kb_end = min(a.k_blocks, kb0 + a.kb_per);
        for (int kb = kb0; kb < kb_end; kb += a.kbs) {
          mbar_wait(smem_u32(&full[s]), ph, abort_flag);
          tc_fence_after();
          // descriptors differ from the stage-0, block-0, k-0 ones only in the start-address field (16-byte units)
          uint64_t da = desc_a0 + (uint64_t)((s * a.stage_bytes) >> 4);
          uint64_t db = desc_b0 + (uint64_t)((s * a.stage_bytes) >> 4);
          for (int kk = 0; kk < a.kbs; ++kk, da += a.a_tile >> 4, db += a.b_tile >> 4) {
#pragma unroll
            for (int k = 0; k < kPtBK / 16; ++k)
              mma_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, ((kb - kb0) | kk | k) != 0);
          }
          mma_commit(smem_u32(&empty[s]));             // frees the stage when these MMAs have read it
          if (++s == NS) { s = 0; ph ^= 1; }
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
      const int tile = item / a.k_split, sp = item - tile * a.k_split;
      const int mt = tile / a.n_tiles, nt = tile - mt * a.n_tiles;
      const int buf = j & 1;
      mbar_wait(smem_u32(&acc_full[buf]), (j >> 1) & 1, abort_flag);
      tc_fence_after();
      const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * a.bn);
      const float* b1 = a.b1 + (size_t)nt * a.bn;
      const float* w2 = a.w2 + (size_t)nt * a.bn;
      const int row = mt * kPtBM + quad * 32 + lane;
      float sum = 0.f;
      if (a.k_split == 1) {
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
      } else {
        // this CTA's range of the hidden dimension: raw sums out, the last range to arrive finishes the unit tile
        float* mine = a.split + (((size_t)nt * a.k_split + sp) * kPtBM + (quad * 32 + lane)) * a.bn;
        for (int c = 0; c < a.bn; c += 32) {
          uint32_t r[32];
          tmem_ld32(t_row + c, r);
          tmem_ld_wait();
          if (row < a.rows) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<uint4*>(mine + c + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
        __threadfence();
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (et == 0) sh_ticket = atomicAdd(&a.split_ticket[nt], 1);
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (sh_ticket != a.k_split - 1) continue;
        __threadfence();
        if (et == 0) a.split_ticket[nt] = 0;
        // all 128 threads share the work: with a short row box several threads take a row, a slice of the unit
        // tile each; a slice's loads (every range, eight columns) go out together, one round trip per eight columns
        const int er = quad * 32 + lane, tpr = kPtBM / a.row_box;
        const int mrow = er % a.row_box, part = er / a.row_box, cw = a.bn / tpr;
        float ps = 0.f;
        if (mrow < a.rows) {
          const float* p0 = a.split + ((size_t)nt * a.k_split * kPtBM + mrow) * a.bn;
          for (int c = part * cw; c < (part + 1) * cw; c += 8) {
            float4 v[kPredKSplit][2];
#pragma unroll
            for (int q = 0; q < kPredKSplit; ++q) {
              if (q < a.k_split) {
                v[q][0] = __ldcg(reinterpret_cast<const float4*>(p0 + (size_t)q * kPtBM * a.bn + c));
                v[q][1] = __ldcg(reinterpret_cast<const float4*>(p0 + (size_t)q * kPtBM * a.bn + c + 4));
              }
            }
            float4 s0 = v[0][0], s1 = v[0][1];
#pragma unroll
            for (int q = 1; q < kPredKSplit; ++q) {
              if (q < a.k_split) {
                s0.x += v[q][0].x; s0.y += v[q][0].y; s0.z += v[q][0].z; s0.w += v[q][0].w;
                s1.x += v[q][1].x; s1.y += v[q][1].y; s1.z += v[q][1].z; s1.w += v[q][1].w;
              }
            }
            ps = fmaf(__ldg(w2 + c), gelu_erf(s0.x + __ldg(b1 + c)), ps);
            ps = fmaf(__ldg(w2 + c + 1), gelu_erf(s0.y + __ldg(b1 + c + 1)), ps);
            ps = fmaf(__ldg(w2 + c + 2), gelu_erf(s0.z + __ldg(b1 + c + 2)), ps);
            ps = fmaf(__ldg(w2 + c + 3), gelu_erf(s0.w + __ldg(b1 + c + 3)), ps);
            ps = fmaf(__ldg(w2 + c + 4), gelu_erf(s1.x + __ldg(b1 + c + 4)), ps);
            ps = fmaf(__ldg(w2 + c + 5), gelu_erf(s1.y + __ldg(b1 + c + 5)), ps);
            ps = fmaf(__ldg(w2 + c + 6), gelu_erf(s1.z + __ldg(b1 + c + 6)), ps);
            ps = fmaf(__ldg(w2 + c + 7), gelu_erf(s1.w + __ldg(b1 + c + 7)), ps);
          }
        }
        sh_red[part][mrow] = ps;
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (part == 0)
          for (int q = 0; q < tpr; ++q) sum += sh_red[q][mrow];
      }
      if (a.n_tiles == 1) {
        if (row < a.rows) pt_emit(a, row, sum + a.b2);
        continue;
      }
      a.partial[(size_t)nt * a.rows_padded + row] = sum;
      __threadfence();
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (et == 0) sh_ticket = atomicAdd(&a.ticket[mt], 1);
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (sh_ticket == a.n_tiles - 1) {
        __threadfence();
        // threads that share a row take a run of unit tiles each; eight loads go out together
        const int er = quad * 32 + lane, tpr = kPtBM / a.row_box;
        const int mrow = er % a.row_box, part = er / a.row_box, tn = (a.n_tiles + tpr - 1) / tpr;
        const int t_end = min(a.n_tiles, (part + 1) * tn);
        const float* pr = a.partial + (size_t)mt * kPtBM + mrow;
        float ps = 0.f;
        for (int t0 = part * tn; t0 < t_end; t0 += 8) {
          float v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = (t0 + i < t_end) ? __ldcg(pr + (size_t)(t0 + i) * a.rows_padded) : 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) ps += v[i];
        }
        sh_red[part][mrow] = ps;
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (part == 0) {
          float tot = 0.f;
          for (int q = 0; q < tpr; ++q) tot += sh_red[q][mrow];
          if (row < a.rows) pt_emit(a, row, tot + a.b2);
        }
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
                                cudaStream_t s, uint8_t* keep, float threshold) {
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
  a.keep = keep; a.threshold = threshold;
  // Few rows (the decode shape, one row per sequence) make this a latency problem: a CTA walks all of the hidden
  // dimension for its 32 units, one dependent DRAM round trip per ring refill.  A row box of 32 or 64 rows
  // instead of 128 shrinks a stage from 20 KB to 8 KB, and the ring takes as many stages as fit (up to 32), so
  // that a third of the walk is in flight at once.
  const int row_box = m_tiles > 1 ? kPtBM : (rows <= 32 ? 32 : (rows <= 64 ? 64 : kPtBM));
  // ... and a copy of a 32 x 64 box costs the producer as much as one of 128 x 64, so a stage of the short form takes
  // four 64-column blocks of the hidden dimension per copy.
  a.kbs = (row_box < kPtBM && a.k_blocks % 4 == 0) ? 4 : 1;
  a.row_box = row_box;
  a.a_tile = row_box * kPtBK * 2;
  a.b_tile = bn * kPtBK * 2;
  a.a_bytes = a.kbs * a.a_tile;
  a.stage_bytes = a.a_bytes + a.kbs * a.b_tile;
  // One row tile: the hidden dimension is cut into ranges (whole stages each) for as many CTAs as the GPU has SMs.
  a.k_split = 1;
  a.kb_per = a.k_blocks;
  if (m_tiles == 1 && ctx->ws.pred_split != nullptr) {
    const int want = std::min({ctx->sm_count / a.n_tiles, kPredKSplit, a.k_blocks / a.kbs});
    if (want > 1) {
      a.kb_per = ((a.k_blocks + want - 1) / want + a.kbs - 1) / a.kbs * a.kbs;
      a.k_split = (a.k_blocks + a.kb_per - 1) / a.kb_per;
    }
  }
  a.split = ctx->ws.pred_split; a.split_ticket = ctx->ws.pred_split_ticket;
  a.stages = std::max(2, std::min({kPtMaxStages, (4 * kPtStageBytes) / a.stage_bytes, a.kb_per / a.kbs}));
  int cols = 32;
  while (cols < 2 * bn) cols <<= 1;
  a.tmem_cols = cols;
  if (m_tiles * kPtBM > a.rows_padded) return cudaErrorInvalidValue;

  CUtensorMap mx, mw;
  // X [rows][hidden] and W1 [units][hidden] seen as (64 columns, row, 64-column block): a box of kbs blocks lands
  // as kbs K-major tiles one after the other
  const uint64_t dx[3] = {(uint64_t)kPtBK, (uint64_t)rows, (uint64_t)a.k_blocks};
  const uint64_t dw[3] = {(uint64_t)kPtBK, (uint64_t)d.pred_hidden, (uint64_t)a.k_blocks};
  const uint64_t st[2] = {(uint64_t)d.hidden * 2, (uint64_t)kPtBK * 2};
  const uint32_t bx[3] = {kPtBK, (uint32_t)row_box, (uint32_t)a.kbs};
  const uint32_t bw[3] = {kPtBK, (uint32_t)bn, (uint32_t)a.kbs};
  if (!encode_bf16_map(ctx->tmap_encode, &mx, x, 3, dx, st, bx) ||
      !encode_bf16_map(ctx->tmap_encode, &mw, p->w1, 3, dw, st, bw))
    return cudaErrorInvalidValue;
  static int attr_set[64];
  if (!attr_set[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(predictor_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPtSmem);
    if (e != cudaSuccess) return e;
    attr_set[ctx->device & 63] = 1;
  }
  const int grid = min(ctx->sm_count, m_tiles * a.n_tiles * a.k_split);
  predictor_tc_kernel<<<grid, kPtThreads, kPtSmem, s>>>(mx, mw, a);
  return cudaGetLastError();
}

}  // namespace dl
