// Compaction of kept rows into the per-sequence cache (set builder of Eq. 5, reduced set of
// Eq. 11, append of Eq. 6).
//
// Source rows are token-major [B][T][H][D]; the cache is head-major [B][H][cap][D], so a kept
// token row of H*D elements lands as H pieces of D elements.  Two kernels:
//   plan : per sequence, count the kept rows, check the capacity, fix the first destination
//          row and (optionally) advance the length;
//   copy : per tile of 32 source tokens, rank the kept ones by a ballot scan on top of the
//          count of kept tokens before the tile, then move each kept row with 16-byte loads
//          and stores (a warp moves 512 contiguous source bytes per instruction).
// Dropped rows are never read.
#include "common.cuh"

namespace dl {

constexpr int kPlanThreads = 256;
constexpr int kCopyThreads = 256;
constexpr int kTileTokens = 32;

__device__ __forceinline__ int block_sum_256(int v, int* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  int t = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) t += sh[w];
  __syncthreads();
  return t;
}

__global__ void __launch_bounds__(kPlanThreads)
compact_plan_kernel(const uint8_t* __restrict__ keep, int32_t keep_cols, const int32_t* __restrict__ t_src, int32_t t_max,
                    int32_t cap, int32_t* __restrict__ cache_len, int32_t commit,
                    int32_t* __restrict__ plan_base, int32_t* __restrict__ plan_count, DeviceStatus* st) {
  __shared__ int sh[8];
  // the copy kernel behind this one may start now: it ranks its tile's tokens first and waits for this
  // kernel's results (grid-dependency wait) only before it needs them
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int b = blockIdx.x;
  int tb = t_src ? t_src[b] : t_max;
  tb = max(0, min(tb, t_max));
  int c = 0;
  if (keep) {
    const uint8_t* kp = keep + (size_t)b * keep_cols;
    for (int i = threadIdx.x; i < tb; i += kPlanThreads) c += (i >= keep_cols || kp[i] != 0);
  } else {
    for (int i = threadIdx.x; i < tb; i += kPlanThreads) c += 1;
  }
  c = block_sum_256(c, sh);
  if (threadIdx.x == 0) {
    int base = cache_len[b];
    if (base < 0 || base + c > cap) {
      report_status(st, DL_ERR_CAPACITY, b);
      plan_base[b] = base;
      plan_count[b] = -1;
    } else {
      plan_base[b] = base;
      plan_count[b] = c;
      if (commit) cache_len[b] = base + c;
    }
  }
}

// v_src == nullptr: one tensor only.  row_units = H*D*elt/16 (16-byte units per token row);
// piece_units = D*elt/16 (units per head piece).
__global__ void __launch_bounds__(kCopyThreads)
compact_copy_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                    const uint8_t* __restrict__ keep, int32_t keep_cols, const int32_t* __restrict__ t_src,
                    int32_t t_max, uint4* __restrict__ k_cache, uint4* __restrict__ v_cache, int32_t cap, int32_t H,
                    int32_t row_units, int32_t piece_units, const int32_t* __restrict__ plan_base,
                    const int32_t* __restrict__ plan_count) {
  __shared__ int sh[8];
  __shared__ int tile_tok[kTileTokens];
  __shared__ int tile_kept;

  const int b = blockIdx.y;
  int tb = t_src ? t_src[b] : t_max;
  tb = max(0, min(tb, t_max));
  const int t0 = blockIdx.x * kTileTokens;
  if (t0 >= tb) return;
  const uint8_t* kp = keep ? keep + (size_t)b * keep_cols : nullptr;

  // kept tokens before this tile
  int before = 0;
  if (kp) {
    for (int i = threadIdx.x; i < t0; i += kCopyThreads) before += (i >= keep_cols || kp[i] != 0);
    before = block_sum_256(before, sh);
  } else {
    before = t0;
  }
  // rank the tile's kept tokens
  if (threadIdx.x < 32) {
    int t = t0 + threadIdx.x;
    bool f = (t < tb) && (kp == nullptr || t >= keep_cols || kp[t] != 0);
    unsigned m = __ballot_sync(0xffffffffu, f);
    if (f) tile_tok[__popc(m & ((1u << threadIdx.x) - 1u))] = t;
    if (threadIdx.x == 0) tile_kept = __popc(m);
  }
  __syncthreads();
  // launched with programmatic stream serialisation: the plan of this call is complete from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (plan_count[b] <= 0) return;
  const int nk = tile_kept;
  const int dst0 = plan_base[b] + before;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_tensors = v_src ? 2 : 1;

  // (token, tensor) pairs are spread over the 8 warps
  for (int job = warp; job < nk * n_tensors; job += kCopyThreads / 32) {
    const int j = job / n_tensors, which = job - j * n_tensors;
    const int t = tile_tok[j];
    const uint4* src = (which ? v_src : k_src) + ((size_t)b * t_max + t) * row_units;
    uint4* dst = (which ? v_cache : k_cache);
    const size_t dst_row = (size_t)(dst0 + j) * piece_units;
    const size_t head_stride = (size_t)cap * piece_units;
    const size_t dst_b = (size_t)b * H * head_stride;
    for (int u0 = 0; u0 < row_units; u0 += 32 * 8) {
      uint4 r[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        int u = u0 + i * 32 + lane;
        if (u < row_units) r[i] = __ldcs(src + u);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        int u = u0 + i * 32 + lane;
        if (u < row_units) {
          int h = u / piece_units, o = u - h * piece_units;
          dst[dst_b + (size_t)h * head_stride + dst_row + o] = r[i];
        }
      }
    }
  }
}

cudaError_t launch_compact(const dl_ctx* ctx, const void* k_src, const void* v_src, const uint8_t* keep,
                           int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                           void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, cudaStream_t s) {
  if (B == 0 || t_src_max == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  const int elt = d.dtype == DL_F32 ? 4 : 2;
  const int piece_units = d.head_dim * elt / 16;
  const int row_units = piece_units * d.n_heads;
  compact_plan_kernel<<<B, kPlanThreads, 0, s>>>(keep, keep_cols, t_src, t_src_max, cap, cache_len, commit,
                                                 ctx->ws.plan_base, ctx->ws.plan_count, ctx->ws.status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 grid((t_src_max + kTileTokens - 1) / kTileTokens, B);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(kCopyThreads); cfg.dynamicSmemBytes = 0; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, compact_copy_kernel, (const uint4*)k_src, (const uint4*)v_src, keep, (int32_t)keep_cols,
                            t_src, (int32_t)t_src_max, (uint4*)k_cache, (uint4*)v_cache, (int32_t)cap, (int32_t)d.n_heads,
                            (int32_t)row_units, (int32_t)piece_units, (const int32_t*)ctx->ws.plan_base,
                            (const int32_t*)ctx->ws.plan_count);
}

__global__ void commit_len_kernel(const uint8_t* __restrict__ keep, int32_t B, int32_t cap,
                                  int32_t* __restrict__ cache_len) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int n = cache_len[b];
  if (keep[b] != 0 && n < cap) cache_len[b] = n + 1;
}

cudaError_t launch_commit_len(const uint8_t* keep, int32_t B, int32_t cap, int32_t* cache_len,
                              cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  commit_len_kernel<<<(B + 127) / 128, 128, 0, s>>>(keep, B, cap, cache_len);
  return cudaGetLastError();
}

}  // namespace dl
