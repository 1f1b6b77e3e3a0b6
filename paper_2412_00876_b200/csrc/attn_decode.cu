// Decode attention over the compacted cache plus the current token (Eq. 6, second line):
//   o = softmax([q.K_cache[0:n) ; q.k_t] * scale) [V_cache[0:n) ; v_t]      per (sequence, head)
// with the conditional append of Eq. 6 fused in (the token's K/V go to row n when keep[b]).
//
// HBM-bound: every cached K and V row is read exactly once.  Design
//   - persistent CTAs (one per SM) walk a list of work items (b, h, chunk of <= CHUNK rows)
//     derived on the device from cache_len, so the launch shape never depends on the lengths;
//   - a producer warp streams 64-row K and V tiles (contiguous in the head-major cache) into a
//     ring of shared-memory stages with bulk asynchronous copies completing on mbarriers;
//   - 8 consumer warps each own 8 rows of a stage: scores with 8 lanes per row and a 3-step
//     shuffle reduction, online softmax kept per warp in registers, P.V with one lane per
//     4 (bf16) or 2 (fp32) output dimensions; the ring runs across item boundaries;
//   - per item the 8 warps' partial (max, sum, acc) are merged through shared memory in a fixed
//     order; sequences longer than one chunk leave partials in the workspace and the CTA that
//     arrives last for a (b, h) merges them in chunk order (a ticket, not a wait), so results
//     are reproducible bit for bit.
// Every mbarrier wait is bounded: when the bound is hit the CTA raises an abort flag, stops
// waiting, drains its outstanding copies and DL_ERR_TIMEOUT is recorded.
#include "common.cuh"
#include "pipeline.cuh"

namespace dl {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumerThreads + 32;   // + producer warp
constexpr int kStageRows = 64;                           // rows of K and of V per stage
constexpr int kRowsPerWarp = kStageRows / kConsumerWarps;
constexpr int kMaxDecodeBatch = 2048;

__device__ __forceinline__ void consumer_bar() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

// ---- unpacking of a 16-byte chunk / a lane's slice into floats -----------------------------
template <typename T> struct Elt;
template <> struct Elt<float> {
  static constexpr int kPerChunk = 4;
  __device__ static __forceinline__ void unpack16(const uint4& c, float* f) {
    f[0] = __uint_as_float(c.x); f[1] = __uint_as_float(c.y);
    f[2] = __uint_as_float(c.z); f[3] = __uint_as_float(c.w);
  }
};
template <> struct Elt<__nv_bfloat16> {
  static constexpr int kPerChunk = 8;
  __device__ static __forceinline__ void unpack16(const uint4& c, float* f) {
    f[0] = bf16lo(c.x); f[1] = bf16hi(c.x); f[2] = bf16lo(c.y); f[3] = bf16hi(c.y);
    f[4] = bf16lo(c.z); f[5] = bf16hi(c.z); f[6] = bf16lo(c.w); f[7] = bf16hi(c.w);
  }
};

// A lane's slice of a row in the P.V phase: LB = row bytes / 32 (4, 8 or 16 bytes).
template <typename T, int LB> struct LaneSlice;
template <> struct LaneSlice<float, 8> {
  static constexpr int kElts = 2;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    float2 v = *reinterpret_cast<const float2*>(p); f[0] = v.x; f[1] = v.y;
  }
};
template <> struct LaneSlice<float, 16> {
  static constexpr int kElts = 4;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
};
template <> struct LaneSlice<__nv_bfloat16, 4> {
  static constexpr int kElts = 2;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    uint32_t v = *reinterpret_cast<const uint32_t*>(p); f[0] = bf16lo(v); f[1] = bf16hi(v);
  }
};
template <> struct LaneSlice<__nv_bfloat16, 8> {
  static constexpr int kElts = 4;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    f[0] = bf16lo(v.x); f[1] = bf16hi(v.x); f[2] = bf16lo(v.y); f[3] = bf16hi(v.y);
  }
};

struct DecodeArgs {
  const void* q; const void* k_t; const void* v_t;
  void* k_cache; void* v_cache;
  const int32_t* cache_len; const uint8_t* keep;
  void* out;
  float* partial; int32_t* ticket; DeviceStatus* status;
  int32_t B, H, cap, chunk, slots, n_stages;
  float scale_log2;
};

template <typename T, int D>
__global__ void __launch_bounds__(kDecodeThreads, 1)
attn_decode_kernel(const DecodeArgs a) {
  constexpr int RB = D * (int)sizeof(T);            // bytes per cache row
  constexpr int NC = RB / 16;                       // 16-byte chunks per row
  constexpr int NCL = NC / 8;                       // chunks per lane in the score phase
  constexpr int EPC = Elt<T>::kPerChunk;
  constexpr int LB = RB / 32;                       // bytes per lane in the P.V phase
  using Slice = LaneSlice<T, LB>;
  constexpr int EPL = Slice::kElts;
  constexpr int TILE_BYTES = kStageRows * RB;       // one K (or V) tile
  constexpr int CW = D + 4;                         // floats per warp slot in the combine buffer
  static_assert(NCL >= 1, "row too short");

  extern __shared__ __align__(128) char smem[];
  char* tiles = smem;                                                     // [n_stages][2][TILE_BYTES]
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + (size_t)a.n_stages * 2 * TILE_BYTES);
  float* comb = reinterpret_cast<float*>(bars + 2 * a.n_stages);         // [2][8][CW]
  int* prefix = reinterpret_cast<int*>(comb + 2 * kConsumerWarps * CW);   // [B + 1]
  __shared__ int sh_abort;
  __shared__ int sh_ticket;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NS = a.n_stages;
  volatile int* abort_flag = &sh_abort;

  // ---- setup: barriers and the item table -------------------------------------------------
  if (tid == 0) {
    sh_abort = 0;
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);                       // full: producer's expect_tx arrive
      mbar_init(smem_u32(&bars[NS + s]), kConsumerWarps);     // empty: one arrive per consumer warp
    }
    fence_mbar_init();
  }
  for (int b = tid; b < a.B; b += kDecodeThreads) {
    int n = min(max(a.cache_len[b], 0), a.cap);
    prefix[b + 1] = max(1, (n + a.chunk - 1) / a.chunk) * a.H;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    prefix[0] = 0;
    for (int b = 0; b < a.B; ++b) { run += prefix[b + 1]; prefix[b + 1] = run; }
  }
  __syncthreads();
  const int total = prefix[a.B];

  auto decode_item = [&](int item, int& b, int& h, int& c, int& nch, int& n_b) {
    int lo = 0, hi = a.B - 1;
    while (lo < hi) {                                   // last b with prefix[b] <= item
      int mid = (lo + hi + 1) >> 1;
      if (prefix[mid] <= item) lo = mid; else hi = mid - 1;
    }
    b = lo;
    n_b = min(max(a.cache_len[b], 0), a.cap);
    nch = max(1, (n_b + a.chunk - 1) / a.chunk);
    int r = item - prefix[b];
    h = r / nch;
    c = r - h * nch;
  };

  if (warp == kConsumerWarps) {
    // =============================== producer warp ===========================================
    if (lane == 0) {
      int it = 0;
      for (int item = blockIdx.x; item < total && !*abort_flag; item += gridDim.x) {
        int b, h, c, nch, n_b;
        decode_item(item, b, h, c, nch, n_b);
        const int r0 = c * a.chunk, rows = min(n_b, r0 + a.chunk) - r0;
        const size_t row0 = ((size_t)(b * a.H + h) * a.cap + r0);
        const char* kg = (const char*)a.k_cache + row0 * RB;
        const char* vg = (const char*)a.v_cache + row0 * RB;
        for (int st = 0; st * kStageRows < rows; ++st, ++it) {
          const int slot = it % NS;
          if (!mbar_wait(smem_u32(&bars[NS + slot]), ((it / NS) & 1) ^ 1, abort_flag)) break;
          const int nr = min(kStageRows, rows - st * kStageRows);
          const uint32_t bytes = (uint32_t)nr * RB;
          const uint32_t full = smem_u32(&bars[slot]);
          mbar_expect_tx(full, 2 * bytes);
          char* dst = tiles + (size_t)slot * 2 * TILE_BYTES;
          bulk_g2s(smem_u32(dst), kg + (size_t)st * TILE_BYTES, bytes, full);
          bulk_g2s(smem_u32(dst + TILE_BYTES), vg + (size_t)st * TILE_BYTES, bytes, full);
        }
      }
      if (*abort_flag) {
        // drain: every stage that was issued must land before the CTA's shared memory is released
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        for (int j = max(0, it - NS); j < it; ++j) {
          const uint32_t full = smem_u32(&bars[j % NS]);
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(full, (j / NS) & 1); ++i) __nanosleep(40);
        }
      }
    }
    return;
  }

  // ================================= consumer warps ===========================================
  const int sub = lane & 7, rg = lane >> 3;
  int it = 0;
  int buf = 0;
  for (int item = blockIdx.x; item < total; item += gridDim.x, buf ^= 1) {
    int b, h, c, nch, n_b;
    decode_item(item, b, h, c, nch, n_b);
    const int r0 = c * a.chunk, rows = min(n_b, r0 + a.chunk) - r0;
    const size_t bh = (size_t)b * a.H + h;

    // query slice of this lane (score-phase layout), pre-scaled by scale * log2(e)
    float qf[NCL][EPC];
    const T* qg = (const T*)a.q + bh * D;
#pragma unroll
    for (int cc = 0; cc < NCL; ++cc) {
      uint4 raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(qg) + (sub + 8 * cc) * 16);
      Elt<T>::unpack16(raw, qf[cc]);
#pragma unroll
      for (int e = 0; e < EPC; ++e) qf[cc][e] *= a.scale_log2;
    }

    float m_run = -INFINITY, l_run = 0.f;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

    for (int st = 0; st * kStageRows < rows; ++st, ++it) {
      const int slot = it % NS;
      mbar_wait(smem_u32(&bars[slot]), (it / NS) & 1, abort_flag);
      const char* Ks = tiles + (size_t)slot * 2 * TILE_BYTES;
      const char* Vs = Ks + TILE_BYTES;
      const int nr = min(kStageRows, rows - st * kStageRows);
      const int vw = min(max(nr - warp * kRowsPerWarp, 0), kRowsPerWarp);   // valid rows of this warp
      if (vw > 0) {
        float s2[2];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          const int lr = p * 4 + rg;
          const char* krow = Ks + (size_t)(warp * kRowsPerWarp + lr) * RB;
          float dot0 = 0.f, dot1 = 0.f;
#pragma unroll
          for (int cc = 0; cc < NCL; ++cc) {
            uint4 raw = *reinterpret_cast<const uint4*>(krow + (sub + 8 * cc) * 16);
            float kf[EPC];
            Elt<T>::unpack16(raw, kf);
#pragma unroll
            for (int e = 0; e < EPC; e += 2) {
              dot0 = fmaf(qf[cc][e], kf[e], dot0);
              dot1 = fmaf(qf[cc][e + 1], kf[e + 1], dot1);
            }
          }
          float dot = dot0 + dot1;
          dot += __shfl_xor_sync(0xffffffffu, dot, 1);
          dot += __shfl_xor_sync(0xffffffffu, dot, 2);
          dot += __shfl_xor_sync(0xffffffffu, dot, 4);
          s2[p] = (lr < vw) ? dot : -INFINITY;
        }
        float mx = fmaxf(s2[0], s2[1]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float m_new = fmaxf(m_run, mx);
        const float corr = exp2f(m_run - m_new);
        const float p0 = exp2f(s2[0] - m_new), p1 = exp2f(s2[1] - m_new);
        float ps = p0 + p1;
        ps += __shfl_xor_sync(0xffffffffu, ps, 8);
        ps += __shfl_xor_sync(0xffffffffu, ps, 16);
        l_run = l_run * corr + ps;
        m_run = m_new;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= corr;
        const char* vrow = Vs + (size_t)(warp * kRowsPerWarp) * RB + lane * LB;
#pragma unroll
        for (int j = 0; j < kRowsPerWarp; ++j) {
          const float pj = __shfl_sync(0xffffffffu, (j < 4) ? p0 : p1, (j & 3) * 8);
          if (j < vw) {
            float vf[EPL];
            Slice::load(vrow + (size_t)j * RB, vf);
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pj, vf[e], acc[e]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[NS + slot]));
    }

    // ---- score of the current token (every 8-lane group computes the same value) ---------------
    float s_e = 0.f;
    {
      const T* kt = (const T*)a.k_t + bh * D;
#pragma unroll
      for (int cc = 0; cc < NCL; ++cc) {
        uint4 raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(kt) + (sub + 8 * cc) * 16);
        float kf[EPC];
        Elt<T>::unpack16(raw, kf);
#pragma unroll
        for (int e = 0; e < EPC; ++e) s_e = fmaf(qf[cc][e], kf[e], s_e);
      }
      s_e += __shfl_xor_sync(0xffffffffu, s_e, 1);
      s_e += __shfl_xor_sync(0xffffffffu, s_e, 2);
      s_e += __shfl_xor_sync(0xffffffffu, s_e, 4);
    }

    // ---- merge the 8 warps of this item (fixed order) ------------------------------------------
    float* cb = comb + (size_t)buf * kConsumerWarps * CW + warp * CW;
#pragma unroll
    for (int e = 0; e < EPL; ++e) cb[lane * EPL + e] = acc[e];
    if (lane == 0) { cb[D] = m_run; cb[D + 1] = l_run; cb[D + 2] = s_e; }
    consumer_bar();
    const float* cball = comb + (size_t)buf * kConsumerWarps * CW;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, cball[w * CW + D]);
    float L = 0.f, A = 0.f;
    if (tid < D) {
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float mw = cball[w * CW + D];
        const float wt = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
        L = fmaf(cball[w * CW + D + 1], wt, L);
        A = fmaf(cball[w * CW + tid], wt, A);
      }
    }
    const float se = cball[D + 2];
    const T* vt = (const T*)a.v_t + bh * D;

    // ---- Eq. 6 append, done once per (b, h) by the item of chunk 0 -----------------------------
    if (c == 0 && a.keep != nullptr && a.keep[b] != 0) {
      if (n_b < a.cap) {
        if (tid < D) {
          const size_t dst = (bh * a.cap + n_b) * D + tid;
          ((T*)a.k_cache)[dst] = ((const T*)a.k_t)[bh * D + tid];
          ((T*)a.v_cache)[dst] = vt[tid];
        }
      } else if (tid == 0 && h == 0) {
        report_status(a.status, DL_ERR_CAPACITY, b);
      }
    }

    if (nch == 1) {
      if (tid < D) {
        const float M2 = fmaxf(M, se);
        const float wc = (M == -INFINITY) ? 0.f : exp2f(M - M2);
        const float we = exp2f(se - M2);
        const float o = (A * wc + we * to_f32<T>(vt[tid])) / (L * wc + we);
        ((T*)a.out)[bh * D + tid] = from_f32<T>(o);
      }
      continue;
    }

    // ---- several chunks: leave a partial, the last CTA to arrive merges all of them --------------
    float* part = a.partial + (bh * a.slots + c) * (size_t)(D + 2);
    if (tid < D) part[tid] = A;
    if (tid == 0) { part[D] = M; part[D + 1] = L; }
    __threadfence();
    consumer_bar();
    if (tid == 0) sh_ticket = atomicAdd(&a.ticket[bh], 1);
    consumer_bar();
    if (sh_ticket == nch - 1) {
      __threadfence();
      const float* p0 = a.partial + bh * a.slots * (size_t)(D + 2);
      float Mg = se;
      for (int cc = 0; cc < nch; ++cc) Mg = fmaxf(Mg, __ldcg(p0 + (size_t)cc * (D + 2) + D));
      if (tid < D) {
        float num = exp2f(se - Mg) * to_f32<T>(vt[tid]);
        float den = exp2f(se - Mg);
        for (int cc = 0; cc < nch; ++cc) {
          const float* pc = p0 + (size_t)cc * (D + 2);
          const float mc = __ldcg(pc + D);
          const float wt = (mc == -INFINITY) ? 0.f : exp2f(mc - Mg);
          num = fmaf(__ldcg(pc + tid), wt, num);
          den = fmaf(__ldcg(pc + D + 1), wt, den);
        }
        ((T*)a.out)[bh * D + tid] = from_f32<T>(num / den);
      }
      if (tid == 0) a.ticket[bh] = 0;
    }
  }
  if (*abort_flag && tid == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
}

template <typename T, int D>
static cudaError_t launch_t(const dl_ctx* ctx, DecodeArgs& a, cudaStream_t s) {
  constexpr int RB = D * (int)sizeof(T);
  constexpr int TILE_BYTES = kStageRows * RB;
  const size_t fixed = 2 * kConsumerWarps * (D + 4) * sizeof(float) + (size_t)(a.B + 1) * sizeof(int) + 256;
  int ns = (int)((ctx->smem_optin - 1024 - (int)fixed) / (2 * TILE_BYTES + 16));
  ns = min(ns, 8);
  if (ns < 2) return cudaErrorInvalidConfiguration;
  a.n_stages = ns;
  const size_t smem = (size_t)ns * 2 * TILE_BYTES + (size_t)ns * 16 + fixed;
  auto kern = attn_decode_kernel<T, D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // one persistent CTA per SM, never more CTAs than the fewest possible items
  int grid = min(ctx->sm_count, a.B * a.H);
  kern<<<grid, kDecodeThreads, smem, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_attn_decode(const dl_ctx* ctx, const void* q, const void* k_t, const void* v_t,
                               void* k_cache, void* v_cache, const int32_t* cache_len,
                               const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                               cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  if (B > kMaxDecodeBatch) return cudaErrorInvalidValue;
  const dl_model_desc& d = ctx->desc;
  DecodeArgs a;
  a.q = q; a.k_t = k_t; a.v_t = v_t; a.k_cache = k_cache; a.v_cache = v_cache;
  a.cache_len = cache_len; a.keep = keep; a.out = out;
  a.partial = ctx->ws.dec_partial; a.ticket = ctx->ws.dec_ticket; a.status = ctx->ws.status;
  a.B = B; a.H = d.n_heads; a.cap = cap;
  int chunk = ctx->opt.decode_chunk > 0 ? ctx->opt.decode_chunk : 256;
  chunk = max(kDecodeMinChunk, (chunk + kStageRows - 1) / kStageRows * kStageRows);
  a.chunk = chunk;
  a.slots = ctx->ws.dec_slots;
  a.n_stages = 0;
  a.scale_log2 = scale * 1.4426950408889634f;
  if (d.dtype == DL_BF16) {
    if (d.head_dim == 128) return launch_t<__nv_bfloat16, 128>(ctx, a, s);
    if (d.head_dim == 64) return launch_t<__nv_bfloat16, 64>(ctx, a, s);
  } else {
    if (d.head_dim == 128) return launch_t<float, 128>(ctx, a, s);
    if (d.head_dim == 64) return launch_t<float, 64>(ctx, a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace dl

// =================================================================================================
// dl_sparse_attn_decode_static: the same kernel for callers that cannot allocate device memory.
//
// Its scratch (split partials and arrival tickets) lives in the fixed array below instead of a
// caller-provided workspace.  Every GPU that loads this library holds the array until the process
// exits.  In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// the address is obtained once per device with cudaGetSymbolAddress while that device is current.
// =================================================================================================
namespace dl {

constexpr size_t kStaticScratchBytes = DL_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_static_ptr[kMaxDevices];       // device address of g_static_scratch, per device (0 = not set up)

// Looks the array's device address up (first call on this device) or returns the cached one.
static cudaError_t static_scratch_for(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  void* p = __atomic_load_n(&g_static_ptr[device], __ATOMIC_ACQUIRE);
  if (p == nullptr) {
    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return e;
    if (prev != device && (e = cudaSetDevice(device)) != cudaSuccess) return e;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess) return e;
    __atomic_store_n(&g_static_ptr[device], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return cudaSuccess;
}

}  // namespace dl

extern "C" int32_t dl_sparse_attn_decode_static(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t,
                                                void* k_cache, void* v_cache, const int32_t* cache_len,
                                                const uint8_t* keep, int32_t B, int32_t cap, float scale,
                                                void* out, void* stream) {
  using namespace dl;
  if (!ctx || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!q_t || !k_t || !v_t || !k_cache || !v_cache || !cache_len || !out) return DL_ERR_INVALID_ARG;
  const uintptr_t all = (uintptr_t)q_t | (uintptr_t)k_t | (uintptr_t)v_t | (uintptr_t)k_cache |
                        (uintptr_t)v_cache | (uintptr_t)out;
  if (all & 15u) return DL_ERR_ALIGNMENT;
  if (B > kMaxDecodeBatch) return DL_ERR_UNSUPPORTED;
  const dl_model_desc& d = ctx->desc;
  int chunk = ctx->opt.decode_chunk > 0 ? ctx->opt.decode_chunk : 256;
  chunk = max(kDecodeMinChunk, (chunk + kStageRows - 1) / kStageRows * kStageRows);
  const int slots = (cap + chunk - 1) / chunk + 1;
  // layout inside the array: tickets [B*H] int32 (256-byte padded) | partials [B*H*slots*(D+2)] float
  const size_t ticket_bytes = ((size_t)B * d.n_heads * sizeof(int32_t) + 255) & ~size_t(255);
  const size_t partial_bytes = (size_t)B * d.n_heads * slots * (d.head_dim + 2) * sizeof(float);
  if (ticket_bytes + partial_bytes > kStaticScratchBytes) return DL_ERR_WORKSPACE;   // beyond the fixed maximum

  void* base = nullptr;
  cudaError_t e = static_scratch_for(ctx->device, &base);
  if (e != cudaSuccess) { ctx->last_cuda = e; return DL_ERR_CUDA; }
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != ctx->device) cudaSetDevice(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the last call left: the tickets must start at zero
  e = cudaMemsetAsync(base, 0, ticket_bytes, s);
  if (e == cudaSuccess) {
    DecodeArgs a;
    a.q = q_t; a.k_t = k_t; a.v_t = v_t; a.k_cache = k_cache; a.v_cache = v_cache;
    a.cache_len = cache_len; a.keep = keep; a.out = out;
    a.ticket = static_cast<int32_t*>(base);
    a.partial = reinterpret_cast<float*>(static_cast<char*>(base) + ticket_bytes);
    a.status = ctx->ws.base ? ctx->ws.status : nullptr;
    a.B = B; a.H = d.n_heads; a.cap = cap; a.chunk = chunk; a.slots = slots; a.n_stages = 0;
    a.scale_log2 = scale * 1.4426950408889634f;
    if (d.dtype == DL_BF16 && d.head_dim == 128) e = launch_t<__nv_bfloat16, 128>(ctx, a, s);
    else if (d.dtype == DL_BF16 && d.head_dim == 64) e = launch_t<__nv_bfloat16, 64>(ctx, a, s);
    else if (d.dtype == DL_F32 && d.head_dim == 128) e = launch_t<float, 128>(ctx, a, s);
    else if (d.dtype == DL_F32 && d.head_dim == 64) e = launch_t<float, 64>(ctx, a, s);
    else e = cudaErrorInvalidValue;
  }
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) { ctx->last_cuda = e; return DL_ERR_CUDA; }
  return DL_OK;
}
