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
#include "pipeline.cuh"

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

// The plan of a call is written by the kernel in front of the copy kernel, which starts while that one
// still runs: its words are read with a load the compiler can neither hoist above the grid-dependency
// wait nor serve from the read-only cache (a pointer marked const __restrict__ invites both).
__device__ __forceinline__ int ld_plan(const int32_t* p) {
  int v;
  asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
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
                    int32_t row_units, int32_t piece_units, const int32_t* plan_base,
                    const int32_t* plan_count) {
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
  if (ld_plan(plan_count + b) <= 0) return;
  const int nk = tile_kept;
  const int dst0 = ld_plan(plan_base + b) + before;
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

// The same copy with bulk (TMA, 1-D) transfers: a kept token row travels global -> shared memory as ONE
// bulk load and leaves as H bulk stores of one head piece each, so no register holds data and a warp keeps
// two rows in flight (the next row loads while this one's pieces are stored).  Four warps per CTA, two row
// buffers per warp in dynamic shared memory.
constexpr int kBulkWarps = 4;

__global__ void __launch_bounds__(kBulkWarps * 32)
compact_copy_bulk_kernel(const char* __restrict__ k_src, const char* __restrict__ v_src,
                         const uint8_t* __restrict__ keep, int32_t keep_cols, const int32_t* __restrict__ t_src,
                         int32_t t_max, char* __restrict__ k_cache, char* __restrict__ v_cache, int32_t cap, int32_t H,
                         int32_t row_bytes, int32_t piece_bytes, const int32_t* plan_base,
                         const int32_t* plan_count, DeviceStatus* st) {
  extern __shared__ __align__(128) char rows_s[];
  __shared__ uint64_t bars[kBulkWarps][2];
  __shared__ int sh[kBulkWarps];
  __shared__ int tile_tok[kTileTokens];
  __shared__ int tile_kept;
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.y;
  int tb = t_src ? t_src[b] : t_max;
  tb = max(0, min(tb, t_max));
  const int t0 = blockIdx.x * kTileTokens;
  if (t0 >= tb) return;
  const uint8_t* kp = keep ? keep + (size_t)b * keep_cols : nullptr;
  if (threadIdx.x == 0) sh_abort = 0;
  if (lane == 0) {
    mbar_init(smem_u32(&bars[warp][0]), 1);
    mbar_init(smem_u32(&bars[warp][1]), 1);
    fence_mbar_init();
  }
  // kept tokens before this tile
  int before = 0;
  if (kp) {
    for (int i = threadIdx.x; i < t0; i += kBulkWarps * 32) before += (i >= keep_cols || kp[i] != 0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    if (lane == 0) sh[warp] = before;
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
  if (kp) {
    before = 0;
#pragma unroll
    for (int w = 0; w < kBulkWarps; ++w) before += sh[w];
  } else {
    before = t0;
  }
  // launched with programmatic stream serialisation: the plan of this call is complete from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (ld_plan(plan_count + b) <= 0) return;
  const int nk = tile_kept;
  const int dst0 = ld_plan(plan_base + b) + before;
  const int n_tensors = v_src ? 2 : 1;
  const int total = nk * n_tensors;
  const int my_jobs = total > warp ? (total - warp + kBulkWarps - 1) / kBulkWarps : 0;
  char* buf = rows_s + (size_t)warp * 2 * row_bytes;
  const size_t head_stride = (size_t)cap * piece_bytes;
  auto load = [&](int idx) {                      // job idx of this warp: (token, tensor) pair warp + idx * warps
    const int job = warp + idx * kBulkWarps;
    const int j = job / n_tensors, which = job - j * n_tensors;
    const char* src = (which ? v_src : k_src) + ((size_t)b * t_max + tile_tok[j]) * row_bytes;
    const uint32_t bar = smem_u32(&bars[warp][idx & 1]);
    mbar_expect_tx(bar, (uint32_t)row_bytes);
    bulk_g2s(smem_u32(buf + (size_t)(idx & 1) * row_bytes), src, (uint32_t)row_bytes, bar);
  };
  int issued = 0;                                 // loads issued so far (the same count in every lane)
  if (my_jobs > 0) {
    if (lane == 0) load(0);
    issued = 1;
  }
  for (int idx = 0; idx < my_jobs; ++idx) {
    if (idx + 1 < my_jobs) {
      // the other buffer held job idx - 1: every lane's stores of it must have read it before it is refilled
      bulk_group_wait_read_all();
      __syncwarp();
      if (lane == 0) load(idx + 1);
      issued = idx + 2;
    }
    const bool ok = mbar_wait(smem_u32(&bars[warp][idx & 1]), (idx >> 1) & 1, abort_flag);
    if (!ok) break;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const int job = warp + idx * kBulkWarps;
    const int j = job / n_tensors, which = job - j * n_tensors;
    char* dst = (which ? v_cache : k_cache) + (size_t)b * H * head_stride + (size_t)(dst0 + j) * piece_bytes;
    const uint32_t src = smem_u32(buf + (size_t)(idx & 1) * row_bytes);
    for (int h = lane; h < H; h += 32) bulk_s2g(dst + (size_t)h * head_stride, src + (uint32_t)(h * piece_bytes), (uint32_t)piece_bytes);
    bulk_group_commit();
  }
  bulk_group_wait_read_all();                     // shared memory is read before the CTA ends
  if (*abort_flag) {
    // a load that was issued must land before the CTA's shared memory is released
    if (lane == 0) {
      report_status(st, DL_ERR_TIMEOUT, blockIdx.y);
      for (int j = max(0, issued - 2); j < issued; ++j)
        for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&bars[warp][j & 1]), (j >> 1) & 1); ++i) __nanosleep(40);
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
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cfg.gridDim = grid; cfg.stream = s;
  // bulk-copy kernel where two row buffers per warp fit the shared memory (they do for every shape at hand:
  // a row is H * D * elt bytes, 8 KB for 32 heads of 128 bf16)
  const size_t row_bytes = (size_t)row_units * 16, bulk_smem = 2 * kBulkWarps * row_bytes;
  if (ctx->opt.compact_impl != 1 && bulk_smem + 1024 <= (size_t)ctx->smem_optin) {
    static int attr_set[64];
    int& set_for = attr_set[ctx->device & 63];
    if (set_for < (int)bulk_smem) {
      e = cudaFuncSetAttribute(compact_copy_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bulk_smem);
      if (e != cudaSuccess) return e;
      set_for = (int)bulk_smem;
    }
    cfg.blockDim = dim3(kBulkWarps * 32); cfg.dynamicSmemBytes = bulk_smem;
    return cudaLaunchKernelEx(&cfg, compact_copy_bulk_kernel, (const char*)k_src, (const char*)v_src, keep,
                              (int32_t)keep_cols, t_src, (int32_t)t_src_max, (char*)k_cache, (char*)v_cache, (int32_t)cap,
                              (int32_t)d.n_heads, (int32_t)row_bytes, (int32_t)(piece_units * 16),
                              (const int32_t*)ctx->ws.plan_base, (const int32_t*)ctx->ws.plan_count, ctx->ws.status);
  }
  cfg.blockDim = dim3(kCopyThreads); cfg.dynamicSmemBytes = 0;
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
