// The paper's own predictors (App. "Details of Predictor Architecture"): a linear layer d -> 512, for the image
// predictor two pre-norm transformer blocks over the image tokens of a sequence (8 heads of 64, hidden 2048),
// and the head 512 -> 256 -> 128 -> 2.  The two outputs per token are the decision values D of Eq. 5: keep iff
// D[:,2] > D[:,1] (argmax); the prefill ranking of Eq. 11 uses the raw D[:,2].
// The dense layers run on the tensor cores (gemm_tc.cu); this file holds what sits between them:
//   layer_norm_kernel   row-wise LayerNorm of the fp32 residual stream into the bf16 operand of the next layer
//                       (or a plain cast), one warp per row;
//   vit_attn_kernel     bidirectional attention among the image tokens of a sequence, 8 heads of 64, on the
//                       warp-level tensor-core instruction (mma.sync m16n8k16): the tcgen05 attention kernel
//                       of this library is built for head_dim 128 and a causal mask, and this one is a small
//                       share of the predictor (the paper puts the whole predictor below 1 % of the model);
//   head_out_kernel     the last layer 128 -> 2, the ranking score D[:,2] and the argmax decision;
// and the host code that runs the chain on caller-provided scratch.
#include <algorithm>

#include "common.cuh"

namespace dl {

constexpr int kPpWidth = DL_PRED2_WIDTH, kPpHeads = 8, kPpHeadDim = 64, kPpMlp = 2048, kPpH1 = 256, kPpH2 = 128;
static_assert(kPpHeads * kPpHeadDim == kPpWidth, "heads");

cudaError_t launch_gemm_tc(const dl_ctx* ctx, const void* A, const void* W, const float* bias, void* out, int M, int N,
                           int K, int ldo, bool out_f32, bool gelu, bool accumulate, cudaStream_t s);
bool gemm_tc_supported(const dl_ctx* ctx);

// ---- LayerNorm (eps 1e-6, biased variance) or plain cast of [rows][512] fp32 -> bf16; one warp per row
__global__ void __launch_bounds__(256)
layer_norm_kernel(const float* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                  __nv_bfloat16* __restrict__ out, int rows) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)row * kPpWidth);
  float4 v[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) v[i] = xr[lane + 32 * i];
  float mean = 0.f, rstd = 1.f;
  if (gamma != nullptr) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    mean = s * (1.0f / kPpWidth);
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, d = v[i].w - mean;
      q += (a * a + b * b) + (c * c + d * d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    rstd = rsqrtf(q * (1.0f / kPpWidth) + 1e-6f);
  }
  uint2* orow = reinterpret_cast<uint2*>(out + (size_t)row * kPpWidth);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float y[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
    if (gamma != nullptr) {
      const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + lane + 32 * i);
      const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + lane + 32 * i);
      y[0] = (y[0] - mean) * rstd * g.x + b.x; y[1] = (y[1] - mean) * rstd * g.y + b.y;
      y[2] = (y[2] - mean) * rstd * g.z + b.z; y[3] = (y[3] - mean) * rstd * g.w + b.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(y[0], y[1]), hi = __floats2bfloat162_rn(y[2], y[3]);
    orow[lane + 32 * i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
}

// ---- attention among the image tokens of one sequence -------------------------------------------------------
// qkv [B * n_max][1536] bf16 (query, key, value projections side by side; head h owns 64 columns of each);
// out [B * n_max][512] bf16.  Grid (query tiles of 64, heads, sequences); 4 warps of 16 query rows.
constexpr int kVaRows = 64, kVaStride = 72;          // tile rows; shared-memory row pitch in elements (144 B: no bank conflicts)

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf162(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

__global__ void __launch_bounds__(128)
vit_attn_kernel(const __nv_bfloat16* __restrict__ qkv, const int32_t* __restrict__ n_vis, int n_max,
                __nv_bfloat16* __restrict__ out, float scale_log2) {
  // K and V tiles are double-buffered: the copies of the next tile run under the arithmetic of this one
  __shared__ __align__(16) __nv_bfloat16 sq[kVaRows * kVaStride], skb[2][kVaRows * kVaStride], svb[2][kVaRows * kVaStride];
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * kVaRows;
  const int n = n_vis ? min(max(n_vis[b], 0), n_max) : n_max;
  if (q0 >= n) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t row_base = (size_t)b * n_max;
  constexpr int LD = 3 * kPpWidth;
  // a [64][64] tile of one of the three projections into shared memory; rows past the sequence read as zero
  auto load_tile = [&](__nv_bfloat16* dst, int r0, int col0) {
    for (int u = tid; u < kVaRows * 8; u += 128) {
      const int r = u >> 3, c = (u & 7) * 8;
      uint4 w = make_uint4(0, 0, 0, 0);
      if (r0 + r < n) w = __ldg(reinterpret_cast<const uint4*>(qkv + (row_base + r0 + r) * LD + col0 + c));
      *reinterpret_cast<uint4*>(dst + r * kVaStride + c) = w;
    }
  };
  // the same tile as asynchronous 16-byte copies (rows past the sequence: zero-filled, from a valid address)
  auto load_tile_async = [&](__nv_bfloat16* dst, int r0, int col0) {
    for (int u = tid; u < kVaRows * 8; u += 128) {
      const int r = u >> 3, c = (u & 7) * 8;
      const bool ok = r0 + r < n;
      const __nv_bfloat16* src = qkv + (row_base + (ok ? r0 + r : 0)) * LD + col0 + c;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst + r * kVaStride + c)),
                   "l"(src), "r"(ok ? 16 : 0) : "memory");
    }
  };
  load_tile(sq, q0, h * kPpHeadDim);
  load_tile_async(skb[0], 0, kPpWidth + h * kPpHeadDim);
  load_tile_async(svb[0], 0, 2 * kPpWidth + h * kPpHeadDim);
  asm volatile("cp.async.commit_group;" ::: "memory");
  __syncthreads();
  // this warp's 16 query rows as A fragments of the four 16-dim steps
  uint32_t qa[4][4];
  {
    const int r = warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      ldsm4((uint32_t)__cvta_generic_to_shared(sq + r * kVaStride + ks * 16 + 8 * (lane >> 4)), qa[ks]);
  }
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};      // rows lane/4 and lane/4 + 8 of the warp's 16

  for (int k0 = 0, it = 0; k0 < n; k0 += kVaRows, ++it) {
    const __nv_bfloat16* sk = skb[it & 1];
    const __nv_bfloat16* sv = svb[it & 1];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                                  // this tile has landed for everyone; the other buffer has been read
    if (k0 + kVaRows < n) {
      load_tile_async(skb[(it + 1) & 1], k0 + kVaRows, kPpWidth + h * kPpHeadDim);
      load_tile_async(svb[(it + 1) & 1], k0 + kVaRows, 2 * kPpWidth + h * kPpHeadDim);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    // S = Q K^T for 64 keys: eight blocks of 8 keys
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int nb = 0; nb < 8; nb += 2) {
        uint32_t kb[4];
        const int key = nb * 8 + (lane & 7) + 8 * (lane >> 4), dim = ks * 16 + 8 * ((lane >> 3) & 1);
        ldsm4((uint32_t)__cvta_generic_to_shared(sk + key * kVaStride + dim), kb);
        mma16816(s[nb], qa[ks], kb[0], kb[1]);
        mma16816(s[nb + 1], qa[ks], kb[2], kb[3]);
      }
    }
    // scale to log2 units, mask the keys past the sequence, online softmax per row
    const int kcol = k0 + 2 * (lane & 3);
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kcol + nb * 8 + (e & 1);
        s[nb][e] = key < n ? s[nb][e] * scale_log2 : -INFINITY;
        mx[e >> 1] = fmaxf(mx[e >> 1], s[nb][e]);
      }
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);                     // finite: key k0 is always a token
      corr[r] = exp2f(m_run[r] - m_new);
      m_run[r] = m_new;
      l_run[r] *= corr[r];
    }
    uint32_t pa[4][4];                                // P as A fragments of the four 16-key steps
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const float p0 = exp2f(s[nb][0] - m_run[0]), p1 = exp2f(s[nb][1] - m_run[0]);
      const float p2 = exp2f(s[nb][2] - m_run[1]), p3 = exp2f(s[nb][3] - m_run[1]);
      l_run[0] += p0 + p1;
      l_run[1] += p2 + p3;
      pa[nb >> 1][(nb & 1) * 2] = pack_bf162(p0, p1);
      pa[nb >> 1][(nb & 1) * 2 + 1] = pack_bf162(p2, p3);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) { o[i][0] *= corr[0]; o[i][1] *= corr[0]; o[i][2] *= corr[1]; o[i][3] *= corr[1]; }
    // O += P V: four 16-key steps, eight blocks of 8 dims
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int nb = 0; nb < 8; nb += 2) {
        uint32_t vb[4];
        const int key = ks * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), dim = nb * 8 + 8 * (lane >> 4);
        ldsm4_t((uint32_t)__cvta_generic_to_shared(sv + key * kVaStride + dim), vb);
        mma16816(o[nb], pa[ks], vb[0], vb[1]);
        mma16816(o[nb + 1], pa[ks], vb[2], vb[3]);
      }
    }
  }
  // the row sums live spread over the four lanes of a row
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const int r_lo = q0 + warp * 16 + (lane >> 2), r_hi = r_lo + 8;
  const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
#pragma unroll
  for (int nb = 0; nb < 8; ++nb) {
    const int col = h * kPpHeadDim + nb * 8 + 2 * (lane & 3);
    if (r_lo < n) *reinterpret_cast<uint32_t*>(out + (row_base + r_lo) * kPpWidth + col) = pack_bf162(o[nb][0] * inv0, o[nb][1] * inv0);
    if (r_hi < n) *reinterpret_cast<uint32_t*>(out + (row_base + r_hi) * kPpWidth + col) = pack_bf162(o[nb][2] * inv1, o[nb][3] * inv1);
  }
}

// ---- last layer 128 -> 2, ranking score and decision; one warp per row ------------------------------------------
// h [rows][128] fp32 (after the second GELU); w3 [2][128], b3 [2].  d_out [rows][2] (may be null), score [rows] =
// D[:,2] (may be null), keep [rows] = D[:,2] > D[:,1] (may be null; NaN drops and is reported).  Rows that are
// padding (index within the sequence >= n_vis[b]) get D = 0, score = -inf, keep = 0.
__global__ void __launch_bounds__(256)
head_out_kernel(const float* __restrict__ h, const float* __restrict__ w3, const float* __restrict__ b3,
                const int32_t* __restrict__ n_vis, int n_max, int rows, float* __restrict__ d_out,
                float* __restrict__ score, uint8_t* __restrict__ keep, DeviceStatus* st) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int b = row / n_max, i = row - b * n_max;
  const bool pad = n_vis != nullptr && i >= n_vis[b];
  const float4 x = reinterpret_cast<const float4*>(h + (size_t)row * kPpH2)[lane];
  const float4 w0 = __ldg(reinterpret_cast<const float4*>(w3) + lane), w1 = __ldg(reinterpret_cast<const float4*>(w3 + kPpH2) + lane);
  float d0 = (x.x * w0.x + x.y * w0.y) + (x.z * w0.z + x.w * w0.w);
  float d1 = (x.x * w1.x + x.y * w1.y) + (x.z * w1.z + x.w * w1.w);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    d0 += __shfl_xor_sync(0xffffffffu, d0, o);
    d1 += __shfl_xor_sync(0xffffffffu, d1, o);
  }
  if (lane != 0) return;
  d0 += __ldg(b3);
  d1 += __ldg(b3 + 1);
  if (pad) { d0 = 0.f; d1 = 0.f; }
  if (d_out) { d_out[2 * (size_t)row] = d0; d_out[2 * (size_t)row + 1] = d1; }
  if (score) score[row] = pad ? -INFINITY : d1;
  if (keep) {
    if (!pad && (d0 != d0 || d1 != d1)) report_status(st, DL_WARN_NAN, row);
    keep[row] = (!pad && d1 > d0) ? 1 : 0;
  }
}

static inline int64_t align256i(int64_t v) { return (v + 255) & ~int64_t(255); }

// scratch layout for `rows` rows: residual stream fp32 | layer input bf16 | wide buffer bf16 (qkv / MLP hidden) |
// attention output bf16 | head hidden bf16 [256] | head hidden fp32 [128]
struct PpScratch { float* r; __nv_bfloat16* xn; __nv_bfloat16* t; __nv_bfloat16* att; __nv_bfloat16* h1; float* h2; int64_t bytes; };
static PpScratch pp_scratch(void* base, int64_t rows) {
  PpScratch s;
  int64_t off = 0;
  auto take = [&](int64_t b) { int64_t o = off; off = align256i(off + b); return static_cast<char*>(base) + o; };
  s.r = reinterpret_cast<float*>(take(rows * kPpWidth * 4));
  s.xn = reinterpret_cast<__nv_bfloat16*>(take(rows * kPpWidth * 2));
  s.t = reinterpret_cast<__nv_bfloat16*>(take(rows * kPpMlp * 2));
  s.att = reinterpret_cast<__nv_bfloat16*>(take(rows * kPpWidth * 2));
  s.h1 = reinterpret_cast<__nv_bfloat16*>(take(rows * kPpH1 * 2));
  s.h2 = reinterpret_cast<float*>(take(rows * kPpH2 * 4));
  s.bytes = off;
  return s;
}
int64_t predictor_paper_scratch_bytes(int64_t rows) { return pp_scratch(nullptr, rows).bytes; }

bool predictor_paper_supported(const dl_ctx* ctx) {
  return ctx->desc.dtype == DL_BF16 && ctx->desc.hidden % 64 == 0 && gemm_tc_supported(ctx);
}

cudaError_t launch_predictor_paper(dl_ctx* ctx, const dl_predictor2* p, const void* x, const int32_t* n_vis, int32_t B,
                                   int32_t n_max, void* scratch, float* d_out, float* score, uint8_t* keep, cudaStream_t s) {
  const int rows = B * n_max;
  if (rows == 0) return cudaSuccess;
  const PpScratch S = pp_scratch(scratch, rows);
  const int d = ctx->desc.hidden;
  const dim3 row_grid((rows + 7) / 8);
  cudaError_t e;
#define DL_TRY(call) do { e = (call); if (e != cudaSuccess) return e; } while (0)
  if (p->n_blocks == 0) {
    // no transformer blocks (the output-text predictor): the projection feeds the head directly
    DL_TRY(launch_gemm_tc(ctx, x, p->in.w, p->in.b, S.xn, rows, kPpWidth, d, kPpWidth, false, false, false, s));
  } else {
    DL_TRY(launch_gemm_tc(ctx, x, p->in.w, p->in.b, S.r, rows, kPpWidth, d, kPpWidth, true, false, false, s));
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)kPpHeadDim);
    for (int i = 0; i < p->n_blocks; ++i) {
      const dl_vit_block& k = p->blocks[i];
      // x = x + Proj(MHA(LN(x)))
      layer_norm_kernel<<<row_grid, 256, 0, s>>>(S.r, k.ln1_g, k.ln1_b, S.xn, rows);
      DL_TRY(cudaGetLastError());
      DL_TRY(launch_gemm_tc(ctx, S.xn, k.qkv.w, k.qkv.b, S.t, rows, 3 * kPpWidth, kPpWidth, 3 * kPpWidth, false, false, false, s));
      vit_attn_kernel<<<dim3((n_max + kVaRows - 1) / kVaRows, kPpHeads, B), 128, 0, s>>>(S.t, n_vis, n_max, S.att, scale_log2);
      DL_TRY(cudaGetLastError());
      DL_TRY(launch_gemm_tc(ctx, S.att, k.proj.w, k.proj.b, S.r, rows, kPpWidth, kPpWidth, kPpWidth, true, false, true, s));
      // x = x + FC2(GELU(FC1(LN(x))))
      layer_norm_kernel<<<row_grid, 256, 0, s>>>(S.r, k.ln2_g, k.ln2_b, S.xn, rows);
      DL_TRY(cudaGetLastError());
      DL_TRY(launch_gemm_tc(ctx, S.xn, k.fc1.w, k.fc1.b, S.t, rows, kPpMlp, kPpWidth, kPpMlp, false, true, false, s));
      DL_TRY(launch_gemm_tc(ctx, S.t, k.fc2.w, k.fc2.b, S.r, rows, kPpWidth, kPpMlp, kPpWidth, true, false, true, s));
    }
    layer_norm_kernel<<<row_grid, 256, 0, s>>>(S.r, nullptr, nullptr, S.xn, rows);        // plain cast for the head
    DL_TRY(cudaGetLastError());
  }
  DL_TRY(launch_gemm_tc(ctx, S.xn, p->h1.w, p->h1.b, S.h1, rows, kPpH1, kPpWidth, kPpH1, false, true, false, s));
  DL_TRY(launch_gemm_tc(ctx, S.h1, p->h2.w, p->h2.b, S.h2, rows, kPpH2, kPpH1, kPpH2, true, true, false, s));
  head_out_kernel<<<row_grid, 256, 0, s>>>(S.h2, p->w3, p->b3, n_vis, n_max, rows, d_out, score, keep,
                                           ctx->ws.base ? ctx->ws.status : nullptr);
  return cudaGetLastError();
#undef DL_TRY
}

}  // namespace dl
