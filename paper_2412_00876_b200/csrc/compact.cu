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
// Dropped rows are never read.  The copy exists in two forms (DL_OPT_COMPACT_IMPL): register-staged by token
// tiles (also the one that reads sources in pinned host memory), and bulk (TMA) copies over even row ranges
// with one tensor store per row, which is the one the library picks where it applies.  Several tensors that
// share one decision (K, V and Q of every layer) are compacted by one plan and a run of copy launches that
// overlap each other's start-up and tail (dl_compact_kv_layers).
#include <algorithm>
#include <cstring>

#include "common.cuh"
#include "pipeline.cuh"
#include "tc05.cuh"

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
                    const int32_t* plan_count, int32_t chained, DeviceStatus* st) {
  __shared__ int sh[8];
  __shared__ int tile_tok[kTileTokens];
  __shared__ int tile_kept;

  const int b = blockIdx.y;
  int tb = t_src ? t_src[b] : t_max;
  tb = max(0, min(tb, t_max));
  const int t0 = blockIdx.x * kTileTokens;
  // A CTA without tokens still waits for the plan kernel before it leaves: a grid whose CTAs all left early
  // would retire before its predecessor, and the next kernel of the stream would no longer be ordered behind
  // the plan's writes.
  if (t0 >= tb) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
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
  // launched with programmatic stream serialisation: the plan of this call is complete from here on (a copy
  // that follows another copy of the same plan need not wait here: its predecessor did; it waits before it ends)
  if (!(chained & 2)) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (chained & 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (ld_plan(plan_count + b) <= 0) {
    if (chained & 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
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
          const size_t at = dst_b + (size_t)h * head_stride + dst_row + o;
          if (DL_IN_BOUNDS(st, KID_COMPACT_COPY, at, (size_t)gridDim.y * H * head_stride)) dst[at] = r[i];
        }
      }
    }
  }
  // completion order inside a run of copies: this one may not end before its predecessor has
  if (chained & 2) asm volatile("griddepcontrol.wait;" ::: "memory");
}

constexpr int kBulkWarps = 4;

// The copy with bulk (TMA) transfers and the work dealt evenly: a kept token row travels global -> shared
// memory as ONE 1-D bulk load and leaves as one tensor store (or H bulk stores of one head piece each), so no
// register holds data and a warp keeps two rows in flight.  The kept rows of the whole batch, in (sequence,
// rank) order, are cut into one contiguous range per CTA (dealing source tokens instead would give a CTA of
// text tokens, all kept, four times the rows of a CTA of vision tokens at a 25 % keep rate).  A CTA reads the
// per-sequence row counts of the plan, finds its range, and for each sequence the range touches ranks the
// sequence's mask once (a block scan over 128 token segments) to list the tokens whose rank falls inside; its
// warps then move those rows, their two-buffer pipelines running on across lists.  Up to 2048 sequences.
constexpr int kRowsList = 64;
constexpr int kRowsMaxBatch = 2048;

// Tensor maps of the two caches for the row stores (32-bit words, no swizzle).
struct RowMaps { alignas(64) unsigned char k[128]; alignas(64) unsigned char v[128]; };

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}

// cache [B*H][cap][piece] as words; box = (piece, 1 row, H heads): what one token row holds, head by head
static bool encode_row_map(void* fn, void* out, const void* base, int piece_bytes, int cap, long long bh, int H) {
  if (!fn || !base) return false;
  if ((piece_bytes & 15) || piece_bytes / 4 > 256 || H > 256) return false;
  cuuint64_t gd[3] = {(cuuint64_t)(piece_bytes / 4), (cuuint64_t)cap, (cuuint64_t)bh};
  cuuint64_t gs[2] = {(cuuint64_t)piece_bytes, (cuuint64_t)piece_bytes * (cuuint64_t)cap};
  cuuint32_t bx[3] = {(cuuint32_t)(piece_bytes / 4), 1u, (cuuint32_t)H};
  cuuint32_t es[3] = {1u, 1u, 1u};
  return reinterpret_cast<EncodeTiledFn>(fn)(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_UINT32, 3,
                                             const_cast<void*>(base), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                             CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Encoding a tensor map costs a few microseconds on the host; the caches of a model come back at every batch,
// so the context remembers the row maps it has built (keyed by base, shape and row pitch).
static bool cached_row_map(const dl_ctx* ctx, void* out, const void* base, int piece_bytes, int cap, long long bh, int H) {
  const long long key_rows = -((long long)cap * 1024 + piece_bytes / 4);    // negative: never equal to a decode map's row count
  for (int i = 0; i < dl_ctx::kMapCache; ++i) {
    const dl_ctx::MapEntry& e = ctx->map_cache[i];
    if (e.base == base && e.rows == key_rows && e.aux == bh) { memcpy(out, e.map, 128); return true; }
  }
  alignas(64) unsigned char tmp[128];
  if (!encode_row_map(ctx->tmap_encode, tmp, base, piece_bytes, cap, bh, H)) return false;
  dl_ctx::MapEntry& e = ctx->map_cache[ctx->map_next];
  memcpy(e.map, tmp, 128);
  e.base = base; e.rows = key_rows; e.aux = bh;
  ctx->map_next = (ctx->map_next + 1) % dl_ctx::kMapCache;
  memcpy(out, tmp, 128);
  return true;
}

__global__ void __launch_bounds__(kBulkWarps * 32)
compact_copy_rows_kernel(const char* __restrict__ k_src, const char* __restrict__ v_src,
                         const uint8_t* __restrict__ keep, int32_t keep_cols, const int32_t* __restrict__ t_src,
                         int32_t t_max, char* __restrict__ k_cache, char* __restrict__ v_cache, int32_t cap, int32_t H,
                         int32_t row_bytes, int32_t piece_bytes, int32_t B, const int32_t* plan_base,
                         const int32_t* plan_count, DeviceStatus* st, const __grid_constant__ RowMaps maps,
                         int32_t use_maps, int32_t chained) {
  extern __shared__ __align__(128) char rows_s[];
  __shared__ uint64_t bars[kBulkWarps][2];
  __shared__ int sh[kBulkWarps];
  __shared__ int s_cnt[kRowsMaxBatch];
  __shared__ int list_tok[kRowsList];
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;
  constexpr int kThreads = kBulkWarps * 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) sh_abort = 0;
  if (lane == 0) {
    mbar_init(smem_u32(&bars[warp][0]), 1);
    mbar_init(smem_u32(&bars[warp][1]), 1);
    fence_mbar_init();
  }
  // Launched with programmatic stream serialisation: the plan of this call is complete from here on.  In a run of
  // copies that share one plan (chained: bit 0 = let the next kernel of the stream start while this one drains,
  // bit 1 = this copy follows another copy of the same plan) only the first waits here; the others started after
  // it had, so the plan is complete for them too, and they wait for their predecessor before they END, which keeps
  // the order of completion that the stream promises to whatever follows the run.
  if (!(chained & 2)) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (chained & 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  int part = 0;
  for (int b = tid; b < B; b += kThreads) {
    const int c = max(ld_plan(plan_count + b), 0);                    // -1: the sequence does not fit, skip it
    s_cnt[b] = c;
    part += c;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0) sh[warp] = part;
  __syncthreads();
  long long n_rows = 0;
#pragma unroll
  for (int w = 0; w < kBulkWarps; ++w) n_rows += sh[w];
  const long long lo = n_rows * blockIdx.x / gridDim.x, hi = n_rows * (blockIdx.x + 1) / gridDim.x;
  if (hi <= lo) {
    if (chained & 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }

  const int n_tensors = v_src ? 2 : 1;
  char* buf = rows_s + (size_t)warp * 2 * row_bytes;
  const size_t head_stride = (size_t)cap * piece_bytes;
  int n_ld = 0;                                   // loads this warp has issued so far (the same in every lane)
  bool ok = true;
  long long off = 0;                              // rows of the sequences before b
  for (int b = 0; b < B && off < hi && ok; ++b) {
    const int cb = s_cnt[b];
    const int ra = (int)max(lo - off, 0LL), rb = (int)min(hi - off, (long long)cb);
    off += cb;
    if (ra >= rb) continue;
    int tb = t_src ? t_src[b] : t_max;
    tb = max(0, min(tb, t_max));
    const uint8_t* kp = keep ? keep + (size_t)b * keep_cols : nullptr;
    const int base_row = ld_plan(plan_base + b);
    const int seg = (tb + kThreads - 1) / kThreads, ts = min(tb, tid * seg), te = min(tb, ts + seg);
    auto kept = [&](int i) { return kp == nullptr || i >= keep_cols || kp[i] != 0; };
    for (int r0 = ra; r0 < rb && ok; r0 += kRowsList) {
      const int r1 = min(rb, r0 + kRowsList);
      // ---- tokens of ranks [r0, r1): block scan of the kept counts of 128 token segments
      int cnt = 0;
      for (int i = ts; i < te; ++i) cnt += kept(i);
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      __syncthreads();                            // the previous list and sh are no longer read
      if (lane == 31) sh[warp] = incl;
      __syncthreads();
      int r = incl - cnt;
      for (int w = 0; w < warp; ++w) r += sh[w];
      if (r < r1 && r + cnt > r0) {
        for (int i = ts; i < te; ++i)
          if (kept(i)) {
            if (r >= r0 && r < r1) list_tok[r - r0] = i;
            ++r;
          }
      }
      __syncthreads();
      // ---- this warp's (row, tensor) jobs of the list: job = warp + idx * warps
      const int total = (r1 - r0) * n_tensors;
      const int my_jobs = total > warp ? (total - warp + kBulkWarps - 1) / kBulkWarps : 0;
      const int dst0 = base_row + r0;
      auto load = [&](int idx) {
        const int job = warp + idx * kBulkWarps;
        const int j = job / n_tensors, which = job - j * n_tensors;
        const char* src = (which ? v_src : k_src) + ((size_t)b * t_max + list_tok[j]) * row_bytes;
        const int g = n_ld + idx;
        const uint32_t bar = smem_u32(&bars[warp][g & 1]);
        mbar_expect_tx(bar, (uint32_t)row_bytes);
        bulk_g2s(smem_u32(buf + (size_t)(g & 1) * row_bytes), src, (uint32_t)row_bytes, bar);
      };
      if (my_jobs > 0) {
        // the buffer's previous row: every lane's stores of it must have read it before it is refilled
        bulk_group_wait_read_all();
        __syncwarp();
        if (lane == 0) load(0);
      }
      int done = 0;
      for (int idx = 0; idx < my_jobs; ++idx) {
        if (idx + 1 < my_jobs) {
          bulk_group_wait_read_all();
          __syncwarp();
          if (lane == 0) load(idx + 1);
        }
        const int g = n_ld + idx;
        done = min(my_jobs, idx + 2);             // loads issued so far in this list
        if (!mbar_wait(smem_u32(&bars[warp][g & 1]), (g >> 1) & 1, abort_flag)) { ok = false; break; }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const int job = warp + idx * kBulkWarps;
        const int j = job / n_tensors, which = job - j * n_tensors;
        char* dst = (which ? v_cache : k_cache) + (size_t)b * H * head_stride + (size_t)(dst0 + j) * piece_bytes;
        const uint32_t src = smem_u32(buf + (size_t)(g & 1) * row_bytes);
        if (use_maps) {
          // the row's H head pieces as ONE tensor store: box (piece, 1 row, H heads) of the cache seen as
          // [B*H][cap][piece]
          if (lane == 0)
            tma_store_3d(reinterpret_cast<const CUtensorMap*>(which ? maps.v : maps.k), src, 0, dst0 + j, b * H);
        } else {
          for (int h = lane; h < H; h += 32) bulk_s2g(dst + (size_t)h * head_stride, src + (uint32_t)(h * piece_bytes), (uint32_t)piece_bytes);
        }
        bulk_group_commit();
      }
      n_ld += ok ? my_jobs : done;
      if (*abort_flag) ok = false;                // another warp gave up: leave together (the loop holds block barriers)
      ok = __syncthreads_and(ok);
    }
  }
  bulk_group_wait_read_all();                     // shared memory is read before the CTA ends
  if (chained & 2) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (*abort_flag) {
    // a load that was issued must land before the CTA's shared memory is released
    if (lane == 0) {
      report_status(st, DL_ERR_TIMEOUT, blockIdx.x);
      for (int j = max(0, n_ld - 2); j < n_ld; ++j)
        for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&bars[warp][j & 1]), (j >> 1) & 1); ++i) __nanosleep(40);
    }
  }
}

// One compaction call: the plan kernel (unless `reuse_plan`: the caller's previous launch in this stream made it
// for the same mask), then the copy.  With `chained` the copy kernel is one of a run of copies that share a
// plan (several layers, one decision): it lets the next one start while it drains and, before it ends, waits for
// its predecessor, so that whatever follows the run finds all of it complete.
cudaError_t launch_compact(const dl_ctx* ctx, const void* k_src, const void* v_src, const uint8_t* keep,
                           int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                           void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, cudaStream_t s,
                           int32_t force_impl, int32_t reuse_plan, int32_t chained) {
  if (B == 0 || t_src_max == 0) return cudaSuccess;
  const int impl = force_impl ? force_impl : ctx->opt.compact_impl;
  const dl_model_desc& d = ctx->desc;
  const int elt = d.dtype == DL_F32 ? 4 : 2;
  const int piece_units = d.head_dim * elt / 16;
  const int row_units = piece_units * d.n_heads;
  cudaError_t e = cudaSuccess;
  if (!reuse_plan) {
    compact_plan_kernel<<<B, kPlanThreads, 0, s>>>(keep, keep_cols, t_src, t_src_max, cap, cache_len, commit,
                                                   ctx->ws.plan_base, ctx->ws.plan_count, ctx->ws.status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  dim3 grid((t_src_max + kTileTokens - 1) / kTileTokens, B);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cfg.gridDim = grid; cfg.stream = s;
  // bulk-copy kernel where two row buffers per warp fit the shared memory (they do for every shape at hand:
  // a row is H * D * elt bytes, 8 KB for 32 heads of 128 bf16) and the batch fits its table of row counts
  const size_t row_bytes = (size_t)row_units * 16, bulk_smem = 2 * kBulkWarps * row_bytes;
  if (impl != 1 && B <= kRowsMaxBatch && bulk_smem + 1024 <= (size_t)ctx->smem_optin) {
    static int attr_set[64];
    int& set_for = attr_set[ctx->device & 63];
    if (set_for < (int)bulk_smem) {
      e = cudaFuncSetAttribute(compact_copy_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bulk_smem);
      if (e != cudaSuccess) return e;
      set_for = (int)bulk_smem;
    }
    cfg.blockDim = dim3(kBulkWarps * 32); cfg.dynamicSmemBytes = bulk_smem;
    // evenly dealt rows: as many CTAs as fit the GPU at once, fewer when the batch has few rows
    const size_t per_cta = bulk_smem + 10 * 1024;
    const long long resident = (long long)ctx->sm_count * std::max<size_t>(1, (size_t)ctx->smem_optin / per_cta);
    const long long by_rows = ((long long)B * t_src_max + 7) / 8;
    cfg.gridDim = dim3((unsigned)std::max(1LL, std::min(resident, by_rows)));
    // one tensor store per row where the row buffers are 128-byte aligned and the maps can be made
    RowMaps maps;
    memset(&maps, 0, sizeof(maps));
    const int piece_bytes = piece_units * 16;
    int32_t use_maps = (row_bytes % 128 == 0) &&
                       cached_row_map(ctx, maps.k, k_cache, piece_bytes, cap, (long long)B * d.n_heads, d.n_heads) &&
                       (!v_src || cached_row_map(ctx, maps.v, v_cache, piece_bytes, cap, (long long)B * d.n_heads, d.n_heads));
    return cudaLaunchKernelEx(&cfg, compact_copy_rows_kernel, (const char*)k_src, (const char*)v_src, keep,
                              (int32_t)keep_cols, t_src, (int32_t)t_src_max, (char*)k_cache, (char*)v_cache,
                              (int32_t)cap, (int32_t)d.n_heads, (int32_t)row_bytes, (int32_t)piece_bytes,
                              (int32_t)B, (const int32_t*)ctx->ws.plan_base, (const int32_t*)ctx->ws.plan_count,
                              ctx->ws.status, maps, use_maps, (int32_t)chained);
  }
  cfg.blockDim = dim3(kCopyThreads); cfg.dynamicSmemBytes = 0;
  return cudaLaunchKernelEx(&cfg, compact_copy_kernel, (const uint4*)k_src, (const uint4*)v_src, keep, (int32_t)keep_cols,
                            t_src, (int32_t)t_src_max, (uint4*)k_cache, (uint4*)v_cache, (int32_t)cap, (int32_t)d.n_heads,
                            (int32_t)row_units, (int32_t)piece_units, (const int32_t*)ctx->ws.plan_base,
                            (const int32_t*)ctx->ws.plan_count, (int32_t)chained, ctx->ws.status);
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
