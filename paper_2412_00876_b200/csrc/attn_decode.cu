// Decode attention over the compacted cache plus the current token (Eq. 6, second line):
//   o = softmax([q.K_cache[0:n) ; q.k_t] * scale) [V_cache[0:n) ; v_t]      per (sequence, head)
// with the conditional append of Eq. 6 fused in (the token's K/V go to row n when keep[b]).
//
// HBM-bound: every cached K and V row is read exactly once.  Design
//   - persistent CTAs (one per SM); the unit of scheduling is a WARP.  Work items (b, h, chunk of
//     <= CHUNK rows) are derived on the device from cache_len and dealt to warps round-robin, so
//     the launch shape never depends on the lengths;
//   - every warp runs its own software pipeline: lane 0 issues bulk asynchronous copies of RS-row
//     K and V tiles (contiguous in the head-major cache) into the warp's private ring of stages,
//     each completing on its own mbarrier; after a stage is consumed its slot is refilled at once,
//     across item boundaries.  No CTA-wide barrier exists in the main loop, so a warp that
//     finishes an item (normalise, write, ticket) never stalls the others;
//   - scores: 8 lanes per row and a 3-step shuffle reduction; online softmax per warp in registers;
//     P.V with one lane per 4 (bf16) or 2 (fp32) output dimensions;
//   - q, k_t, v_t of the NEXT item are fetched into registers while the current one streams;
//   - sequences longer than one chunk leave (max, sum, acc) partials in the scratch and the warp
//     that arrives last for a (b, h) merges them in chunk order (a ticket, not a wait), so results
//     are reproducible bit for bit.
// Every mbarrier wait is bounded: when the bound is hit the CTA raises an abort flag, stops
// waiting and issuing, drains its outstanding copies and DL_ERR_TIMEOUT is recorded.
#include <string.h>

#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kMaxDecodeBatch = 2048;
constexpr int kDecodeRowAlign = 64;      // chunk sizes are multiples of this

// ---- unpacking of a 16-byte chunk into floats ------------------------------------------------
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

// ---- a lane's slice of a row in the P.V phase: LB = row bytes / 32 (4, 8 or 16 bytes) -----------
template <typename T, int LB> struct LaneSlice;
template <> struct LaneSlice<float, 8> {
  using Raw = uint2; static constexpr int kElts = 2;
  __device__ static __forceinline__ void unpack(Raw v, float* f) { f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); }
  __device__ static __forceinline__ Raw pack(const float* f) { return make_uint2(__float_as_uint(f[0]), __float_as_uint(f[1])); }
};
template <> struct LaneSlice<float, 16> {
  using Raw = uint4; static constexpr int kElts = 4;
  __device__ static __forceinline__ void unpack(Raw v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ Raw pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}
template <> struct LaneSlice<__nv_bfloat16, 4> {
  using Raw = uint32_t; static constexpr int kElts = 2;
  __device__ static __forceinline__ void unpack(Raw v, float* f) { f[0] = bf16lo(v); f[1] = bf16hi(v); }
  __device__ static __forceinline__ Raw pack(const float* f) { return pack_bf16x2(f[0], f[1]); }
};
template <> struct LaneSlice<__nv_bfloat16, 8> {
  using Raw = uint2; static constexpr int kElts = 4;
  __device__ static __forceinline__ void unpack(Raw v, float* f) {
    f[0] = bf16lo(v.x); f[1] = bf16hi(v.x); f[2] = bf16lo(v.y); f[3] = bf16hi(v.y);
  }
  __device__ static __forceinline__ Raw pack(const float* f) { return make_uint2(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3])); }
};

struct DecodeArgs {
  const void* q; const void* k_t; const void* v_t;
  void* k_cache; void* v_cache;
  const int32_t* cache_len; const uint8_t* keep;
  void* out;
  float* partial; int32_t* ticket; DeviceStatus* status;
  int32_t B, H, cap, chunk, per_bh, slots, n_stages;
  int32_t* commit_len;    // not null: this launch is the last of a step; it closes the step with cache_len[b] += keep[b]
  int32_t* commit_count;  // CTAs of this launch that have finished (zero between launches)
  int32_t overlap;        // launched with programmatic stream serialisation (see launch_mma)
  int32_t one_slot;       // host only: one CTA per SM (see launch_attn_decode)
  float scale_log2;
};

// Work items of a sequence with n cached rows: an explicit chunk size wins; otherwise up to per_bh
// items of at least kDecodeMinChunk rows each (per_bh is chosen on the host so that the items of
// the whole batch roughly equal the number of warps in the grid).
__device__ __forceinline__ int decode_chunks(int n, const DecodeArgs& a) {
  if (a.chunk > 0) return max(1, (n + a.chunk - 1) / a.chunk);
  return max(1, min(a.per_bh, n / kDecodeMinChunk));
}

static inline int max_chunks(const DecodeArgs& a) {
  return a.chunk > 0 ? (a.cap + a.chunk - 1) / a.chunk : max(1, min(a.per_bh, a.cap / kDecodeMinChunk));
}

struct DecodeItem { int b, h, c, nch, n_b, r0, rows, nst; };

// Closes a decode step inside its last attention launch (Eq. 6: the length grows by the decision, once, after
// every layer has appended): the CTA that finishes last - every other CTA of this launch has read the lengths
// for the last time, and every earlier layer's launch is complete - advances them.  Called by all threads.
__device__ __forceinline__ void decode_commit(const DecodeArgs& a) {
  if (a.commit_len == nullptr) return;
  __shared__ int sh_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    sh_last = atomicAdd(a.commit_count, 1) == (int)gridDim.x - 1;
  }
  __syncthreads();
  if (!sh_last) return;
  for (int b = threadIdx.x; b < a.B; b += blockDim.x) {
    const int n = a.commit_len[b];
    if (a.keep[b] != 0 && n < a.cap) a.commit_len[b] = n + 1;
  }
  if (threadIdx.x == 0) *a.commit_count = 0;
}

template <typename T, int D, int RS, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 1)
attn_decode_kernel(const DecodeArgs a) {
  constexpr int RB = D * (int)sizeof(T);            // bytes per cache row
  constexpr int NC = RB / 16;                       // 16-byte chunks per row
  constexpr int NCL = NC / 8;                       // chunks per lane in the score phase
  constexpr int EPC = Elt<T>::kPerChunk;
  constexpr int LB = RB / 32;                       // bytes per lane in the P.V phase
  using Slice = LaneSlice<T, LB>;
  using Raw = typename Slice::Raw;
  constexpr int EPL = Slice::kElts;
  constexpr int P = RS / 4;                         // score passes per stage (4 rows per pass)
  constexpr int TILE = RS * RB;                     // one K (or V) tile
  static_assert(NCL >= 1 && RS % 4 == 0, "bad tile shape");

  extern __shared__ __align__(128) char smem[];
  const int NS = a.n_stages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  char* my_tiles = smem + (size_t)warp * NS * 2 * TILE;                              // [NS][2][TILE]
  uint64_t* all_bars = reinterpret_cast<uint64_t*>(smem + (size_t)WARPS * NS * 2 * TILE);
  uint64_t* bars = all_bars + warp * NS;
  int* prefix = reinterpret_cast<int*>(all_bars + WARPS * NS);                       // [B + 1]
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;

  // ---- setup: barriers and the item table --------------------------------------------------------
  if (tid == 0) sh_abort = 0;
  if (lane == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_mbar_init();
  }
  for (int b = tid; b < a.B; b += WARPS * 32) {
    int n = min(max(a.cache_len[b], 0), a.cap);
    prefix[b + 1] = decode_chunks(n, a) * a.H;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    prefix[0] = 0;
    for (int b = 0; b < a.B; ++b) { run += prefix[b + 1]; prefix[b + 1] = run; }
  }
  __syncthreads();
  const int total = prefix[a.B];
  // with fewer items than warps the items are dealt across the SMs first; otherwise a CTA's warps
  // take neighbouring items (neighbouring memory)
  const int GW = gridDim.x * WARPS;
  const int gw = (total >= GW) ? blockIdx.x * WARPS + warp : warp * gridDim.x + blockIdx.x;

  auto load_item = [&](int item, DecodeItem& I) {
    int lo = 0, hi = a.B - 1;
    while (lo < hi) {                                   // last b with prefix[b] <= item
      int mid = (lo + hi + 1) >> 1;
      if (prefix[mid] <= item) lo = mid; else hi = mid - 1;
    }
    I.b = lo;
    I.n_b = min(max(a.cache_len[lo], 0), a.cap);
    I.nch = decode_chunks(I.n_b, a);
    const int r = item - prefix[lo];
    I.h = r / I.nch;
    I.c = r - I.h * I.nch;
    // the sequence's rows are split evenly over its chunks, in whole stages
    const int cs = ((I.n_b + I.nch - 1) / I.nch + RS - 1) / RS * RS;
    I.r0 = I.c * cs;
    I.rows = max(0, min(I.n_b, I.r0 + cs) - I.r0);
    I.nst = max(1, (I.rows + RS - 1) / RS);
  };
  // lane 0: fill `slot` with stage `st` of item I (an item without rows still completes one phase)
  auto issue = [&](const DecodeItem& I, int st, int slot) {
    const uint32_t full = smem_u32(&bars[slot]);
    const int nr = min(RS, I.rows - st * RS);
    if (nr <= 0) { mbar_arrive(full); return; }
    const size_t row0 = ((size_t)(I.b * a.H + I.h) * a.cap + (size_t)I.r0 + (size_t)st * RS);
    const uint32_t bytes = (uint32_t)nr * RB;
    mbar_expect_tx(full, 2 * bytes);
    char* dst = my_tiles + (size_t)slot * 2 * TILE;
    bulk_g2s(smem_u32(dst), (const char*)a.k_cache + row0 * RB, bytes, full);
    bulk_g2s(smem_u32(dst + TILE), (const char*)a.v_cache + row0 * RB, bytes, full);
  };

  // ---- producer cursor and prologue ----------------------------------------------------------------
  int p_item = gw, p_st = 0, issued = 0, consumed = 0;
  DecodeItem PI;
  bool p_valid = p_item < total;
  if (p_valid) load_item(p_item, PI);
  auto advance_producer = [&]() {
    ++issued;
    if (++p_st == PI.nst) {
      p_st = 0;
      p_item += GW;
      p_valid = p_item < total;
      if (p_valid) load_item(p_item, PI);
    }
  };
  while (issued < NS && p_valid) {
    if (lane == 0) issue(PI, p_st, issued % NS);
    advance_producer();
  }

  // ---- registers fetched one item ahead: q and k_t (score layout), k_t and v_t (slice layout) ---------
  const int sub = lane & 7, rg = lane >> 3;
  uint4 nq[NCL], nk[NCL];
  Raw nks, nvs;
  auto prefetch = [&](const DecodeItem& I) {
    const size_t off = ((size_t)I.b * a.H + I.h) * RB;
#pragma unroll
    for (int cc = 0; cc < NCL; ++cc) {
      nq[cc] = __ldg(reinterpret_cast<const uint4*>((const char*)a.q + off + (sub + 8 * cc) * 16));
      nk[cc] = __ldg(reinterpret_cast<const uint4*>((const char*)a.k_t + off + (sub + 8 * cc) * 16));
    }
    nks = __ldg(reinterpret_cast<const Raw*>((const char*)a.k_t + off + lane * LB));
    nvs = __ldg(reinterpret_cast<const Raw*>((const char*)a.v_t + off + lane * LB));
  };
  DecodeItem I, NI;
  if (gw < total) { load_item(gw, NI); prefetch(NI); }

  for (int item = gw; item < total; item += GW) {
    I = NI;
    const size_t bh = (size_t)I.b * a.H + I.h;
    // ---- this item's query (pre-scaled by scale*log2 e), current-token score and value slice
    float qf[NCL][EPC];
    float s_e = 0.f;
#pragma unroll
    for (int cc = 0; cc < NCL; ++cc) {
      float kf[EPC];
      Elt<T>::unpack16(nq[cc], qf[cc]);
      Elt<T>::unpack16(nk[cc], kf);
#pragma unroll
      for (int e = 0; e < EPC; ++e) { qf[cc][e] *= a.scale_log2; s_e = fmaf(qf[cc][e], kf[e], s_e); }
    }
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 1);
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 2);
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 4);
    float vt[EPL];
    Slice::unpack(nvs, vt);
    // ---- Eq. 6 append, once per (b, h): the item of chunk 0 writes the token's K/V to row n_b
    if (I.c == 0 && a.keep != nullptr && a.keep[I.b] != 0) {
      if (I.n_b < a.cap) {
        const size_t dst = (bh * a.cap + I.n_b) * RB + lane * LB;
        *reinterpret_cast<Raw*>((char*)a.k_cache + dst) = nks;
        *reinterpret_cast<Raw*>((char*)a.v_cache + dst) = nvs;
      } else if (lane == 0 && I.h == 0) {
        report_status(a.status, DL_ERR_CAPACITY, I.b);
      }
    }
    if (item + GW < total) { load_item(item + GW, NI); prefetch(NI); }

    float m_run = -INFINITY, l_run = 0.f;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

    for (int st = 0; st < I.nst; ++st, ++consumed) {
      const int slot = consumed % NS;
      mbar_wait(smem_u32(&bars[slot]), (consumed / NS) & 1, abort_flag);
      const char* Ks = my_tiles + (size_t)slot * 2 * TILE;
      const char* Vs = Ks + TILE;
      const int nr = min(RS, I.rows - st * RS);
      if (nr > 0) {
        float s[P];
#pragma unroll
        for (int p = 0; p < P; ++p) {
          const int lr = p * 4 + rg;
          const char* krow = Ks + (size_t)lr * RB;
          float dot0 = 0.f, dot1 = 0.f;
#pragma unroll
          for (int cc = 0; cc < NCL; ++cc) {
            const uint4 raw = *reinterpret_cast<const uint4*>(krow + (sub + 8 * cc) * 16);
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
          s[p] = (lr < nr) ? dot : -INFINITY;
        }
        float mx = s[0];
#pragma unroll
        for (int p = 1; p < P; ++p) mx = fmaxf(mx, s[p]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float m_new = fmaxf(m_run, mx);
        const float corr = exp2f(m_run - m_new);
        float ps = 0.f;
#pragma unroll
        for (int p = 0; p < P; ++p) { s[p] = exp2f(s[p] - m_new); ps += s[p]; }
        ps += __shfl_xor_sync(0xffffffffu, ps, 8);
        ps += __shfl_xor_sync(0xffffffffu, ps, 16);
        l_run = l_run * corr + ps;
        m_run = m_new;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= corr;
        const char* vrow = Vs + lane * LB;
#pragma unroll
        for (int j = 0; j < RS; ++j) {
          const float pj = __shfl_sync(0xffffffffu, s[j >> 2], (j & 3) * 8);
          if (j < nr) {
            float vf[EPL];
            Slice::unpack(*reinterpret_cast<const Raw*>(vrow + (size_t)j * RB), vf);
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pj, vf[e], acc[e]);
          }
        }
      }
      __syncwarp();
      // the slot is free again: refill it with the next stage of this warp's stream
      if (p_valid && !*abort_flag) {
        if (lane == 0) issue(PI, p_st, slot);
        advance_producer();
      }
    }

    // ---- finish the item ---------------------------------------------------------------------------
    if (I.nch == 1) {
      const float M2 = fmaxf(m_run, s_e);
      const float wc = (m_run == -INFINITY) ? 0.f : exp2f(m_run - M2);
      const float we = exp2f(s_e - M2);
      const float inv = 1.f / (l_run * wc + we);
      float o[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[e] = (acc[e] * wc + we * vt[e]) * inv;
      *reinterpret_cast<Raw*>((char*)a.out + bh * RB + lane * LB) = Slice::pack(o);
      continue;
    }
    // several chunks: leave a partial; the warp that arrives last merges all of them in chunk order
    float* part = a.partial + (bh * a.slots + I.c) * (size_t)(D + 2);
#pragma unroll
    for (int e = 0; e < EPL; ++e) part[lane * EPL + e] = acc[e];
    if (lane == 0) { part[D] = m_run; part[D + 1] = l_run; }
    __threadfence();
    __syncwarp();
    int ticket = 0;
    if (lane == 0) ticket = atomicAdd(&a.ticket[bh], 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket == I.nch - 1) {
      __threadfence();
      const float* p0 = a.partial + bh * a.slots * (size_t)(D + 2);
      float Mg = s_e;
      for (int cc = 0; cc < I.nch; ++cc) Mg = fmaxf(Mg, __ldcg(p0 + (size_t)cc * (D + 2) + D));
      const float we = exp2f(s_e - Mg);
      float num[EPL];
      float den = we;
#pragma unroll
      for (int e = 0; e < EPL; ++e) num[e] = we * vt[e];
      for (int cc = 0; cc < I.nch; ++cc) {
        const float* pc = p0 + (size_t)cc * (D + 2);
        const float mc = __ldcg(pc + D);
        const float wt = (mc == -INFINITY) ? 0.f : exp2f(mc - Mg);
        den = fmaf(__ldcg(pc + D + 1), wt, den);
#pragma unroll
        for (int e = 0; e < EPL; ++e) num[e] = fmaf(__ldcg(pc + lane * EPL + e), wt, num[e]);
      }
      const float inv = 1.f / den;
#pragma unroll
      for (int e = 0; e < EPL; ++e) num[e] *= inv;
      *reinterpret_cast<Raw*>((char*)a.out + bh * RB + lane * LB) = Slice::pack(num);
      if (lane == 0) a.ticket[bh] = 0;
    }
  }

  if (*abort_flag) {
    // every copy that was issued must land before the CTA's shared memory is released
    if (lane == 0) {
      report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
      for (int j = max(0, issued - NS); j < issued; ++j)
        for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&bars[j % NS]), (j / NS) & 1); ++i) __nanosleep(40);
    }
  }
  decode_commit(a);
}

template <typename T, int D, int RS, int WARPS>
static cudaError_t launch_cfg(const dl_ctx* ctx, DecodeArgs& a, cudaStream_t s) {
  constexpr int RB = D * (int)sizeof(T);
  constexpr int TILE = RS * RB;
  const size_t fixed = (size_t)(a.B + 1) * sizeof(int) + 512;
  int ns = (int)((ctx->smem_optin - (int)fixed) / (WARPS * (2 * TILE + 8)));
  ns = min(ns, 8);
  if (ns < 2) return cudaErrorInvalidConfiguration;
  a.n_stages = ns;
  const size_t smem = (size_t)WARPS * ns * (2 * TILE + 8) + fixed;
  auto kern = attn_decode_kernel<T, D, RS, WARPS>;
  static int attr_set[64];                           // opt-in shared memory size, set once per device and size
  int& attr_set_for = attr_set[ctx->device & 63];
  if (attr_set_for != (int)smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set_for = (int)smem;
  }
  // one persistent CTA per SM, never more CTAs than there can be items
  const long long max_items = (long long)a.B * a.H * max_chunks(a);
  const int grid = (int)max(1LL, min((long long)ctx->sm_count, max_items));
  kern<<<grid, WARPS * 32, smem, s>>>(a);
  return cudaGetLastError();
}

// =================================================================================================
// bf16, head_dim 128: the same warp-private pipeline with the two contractions on the warp-level
// tensor-core instruction (mma.sync m16n8k16).  The CUDA-core kernel above spends ~100 instructions
// per KB of cache and is issue-bound at about 40 % of the HBM rate; here a 16-row tile (8 KB of K
// and V) costs 32 MMAs + 16 ldmatrix + a few dozen softmax instructions.  The query occupies row 0
// of the 16-row A operand (the other rows are zero), K rows are the B operand of q.K^T, the
// probabilities (bf16) are the A operand and V (loaded transposed) the B operand of P.V.
// Tiles are fetched with TMA tile copies using the 128-byte swizzle so that ldmatrix is free of
// bank conflicts; each 16-row tile is four 2 KB boxes (K low/high 64 dims, V low/high 64 dims).
// =================================================================================================
constexpr int kMmaWarps = 4;                      // warps per CTA
constexpr int kMmaCtas = 2;                       // CTAs per SM: with overlapped launches a CTA of the next
                                                  // layer moves in as soon as one of the two has finished
constexpr int kMmaRows = 16;                       // rows per stage
constexpr int kMmaBox = kMmaRows * 128;            // one box: 16 rows x 64 bf16
constexpr int kMmaStage = 4 * kMmaBox;             // K lo | K hi | V lo | V hi

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D += A(16x16, only rows 0-7 of the fragment can be non-zero here) * B(16x8)
__device__ __forceinline__ void mma_16816(float* c, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void tma_tile_2d(uint32_t dst, const void* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

struct TmapPair { alignas(64) unsigned char k[128]; alignas(64) unsigned char v[128]; };

__global__ void __launch_bounds__(kMmaWarps * 32, kMmaCtas)
attn_decode_mma_kernel(const __grid_constant__ TmapPair maps, const DecodeArgs a) {
  constexpr int D = 128, RB = 256, RS = kMmaRows;
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NS = a.n_stages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  char* my_tiles = smem + (size_t)warp * NS * kMmaStage;
  uint64_t* all_bars = reinterpret_cast<uint64_t*>(smem + (size_t)kMmaWarps * NS * kMmaStage);
  uint64_t* bars = all_bars + warp * NS;
  int* prefix = reinterpret_cast<int*>(all_bars + kMmaWarps * NS);
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;

  // Let the next kernel of the stream start as soon as SMs free up (it only matters when that kernel
  // was launched with programmatic stream serialisation; a no-op otherwise).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) sh_abort = 0;
  if (lane == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_mbar_init();
  }
  for (int b = tid; b < a.B; b += kMmaWarps * 32) {
    int n = min(max(a.cache_len[b], 0), a.cap);
    prefix[b + 1] = decode_chunks(n, a) * a.H;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    prefix[0] = 0;
    for (int b = 0; b < a.B; ++b) { run += prefix[b + 1]; prefix[b + 1] = run; }
  }
  __syncthreads();
  const int total = prefix[a.B];
  const int GW = gridDim.x * kMmaWarps;
  const int gw = (total >= GW) ? blockIdx.x * kMmaWarps + warp : warp * gridDim.x + blockIdx.x;

  auto load_item = [&](int item, DecodeItem& I) {
    int lo = 0, hi = a.B - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (prefix[mid] <= item) lo = mid; else hi = mid - 1;
    }
    I.b = lo;
    I.n_b = min(max(a.cache_len[lo], 0), a.cap);
    I.nch = decode_chunks(I.n_b, a);
    const int r = item - prefix[lo];
    I.h = r / I.nch;
    I.c = r - I.h * I.nch;
    const int cs = ((I.n_b + I.nch - 1) / I.nch + RS - 1) / RS * RS;
    I.r0 = I.c * cs;
    I.rows = max(0, min(I.n_b, I.r0 + cs) - I.r0);
    I.nst = max(1, (I.rows + RS - 1) / RS);
  };
  // lane 0: whole 16-row boxes are fetched even for a ragged last tile (the surplus rows are
  // masked); rows past the end of the tensor read as zero
  auto issue = [&](const DecodeItem& I, int st, int slot) {
    const uint32_t full = smem_u32(&bars[slot]);
    if (I.rows - st * RS <= 0) { mbar_arrive(full); return; }
    const int row0 = (I.b * a.H + I.h) * a.cap + I.r0 + st * RS;
    mbar_expect_tx(full, kMmaStage);
    const uint32_t dst = smem_u32(my_tiles + (size_t)slot * kMmaStage);
    tma_tile_2d(dst, maps.k, 0, row0, full);
    tma_tile_2d(dst + kMmaBox, maps.k, 64, row0, full);
    tma_tile_2d(dst + 2 * kMmaBox, maps.v, 0, row0, full);
    tma_tile_2d(dst + 3 * kMmaBox, maps.v, 64, row0, full);
  };

  int p_item = gw, p_st = 0, issued = 0, consumed = 0;
  DecodeItem PI;
  bool p_valid = p_item < total;
  if (p_valid) load_item(p_item, PI);
  auto advance_producer = [&]() {
    ++issued;
    if (++p_st == PI.nst) {
      p_st = 0;
      p_item += GW;
      p_valid = p_item < total;
      if (p_valid) load_item(p_item, PI);
    }
  };
  while (issued < NS && p_valid) {
    if (lane == 0) issue(PI, p_st, issued % NS);
    advance_producer();
  }

  // ---- registers fetched one item ahead.  Fragment layout: lane t (< 4) owns, for each 16-dim
  //      block ks, the 32-bit words ks*8 + t and ks*8 + 4 + t of a row (dims 16ks+2t.. and 16ks+8+2t..)
  const int t4 = lane & 3;
  const bool row0_lane = lane < 4;
  uint32_t nq[16], nk[16];
  uint2 nks, nvs;                                     // raw 8-byte slices for the append
  auto prefetch = [&](const DecodeItem& I) {
    const size_t off = ((size_t)I.b * a.H + I.h) * RB;
    const uint32_t* qw = reinterpret_cast<const uint32_t*>((const char*)a.q + off);
    const uint32_t* kw = reinterpret_cast<const uint32_t*>((const char*)a.k_t + off);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int w = (i >> 1) * 8 + (i & 1) * 4 + t4;
      nq[i] = row0_lane ? __ldg(qw + w) : 0u;
      nk[i] = row0_lane ? __ldg(kw + w) : 0u;
    }
    nks = __ldg(reinterpret_cast<const uint2*>((const char*)a.k_t + off + lane * 8));
    nvs = __ldg(reinterpret_cast<const uint2*>((const char*)a.v_t + off + lane * 8));
  };
  DecodeItem I, NI;
  if (gw < total) { load_item(gw, NI); prefetch(NI); }

  // ldmatrix lane addressing (row within the 16-row tile, 16-byte chunk selector)
  const int k_row = (lane & 7) + ((lane >> 4) << 3);  // q.K^T: matrices 0,1 rows 0-7; 2,3 rows 8-15
  const int k_csel = (lane >> 3) & 1;                 //        matrices 0,2 first chunk; 1,3 second
  const int v_row = (lane & 7) + (((lane >> 3) & 1) << 3);   // P.V: matrices 0,2 rows 0-7; 1,3 rows 8-15
  const int v_csel = lane >> 4;                               //      matrices 0,1 first chunk; 2,3 second

  for (int item = gw; item < total; item += GW) {
    I = NI;
    const size_t bh = (size_t)I.b * a.H + I.h;
    uint32_t qa[16];
    float s_e = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      qa[i] = nq[i];
      s_e = fmaf(bf16lo(nq[i]), bf16lo(nk[i]), s_e);
      s_e = fmaf(bf16hi(nq[i]), bf16hi(nk[i]), s_e);
    }
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 1);
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 2);
    s_e = __shfl_sync(0xffffffffu, s_e, 0) * a.scale_log2;
    if (I.c == 0 && a.keep != nullptr && a.keep[I.b] != 0) {
      if (I.n_b < a.cap) {
        const size_t dst = (bh * a.cap + I.n_b) * RB + lane * 8;
        if (DL_IN_BOUNDS(a.status, KID_DECODE_MMA, dst + 7, (size_t)a.B * a.H * a.cap * RB)) {
          *reinterpret_cast<uint2*>((char*)a.k_cache + dst) = nks;
          *reinterpret_cast<uint2*>((char*)a.v_cache + dst) = nvs;
        }
      } else if (lane == 0 && I.h == 0) {
        report_status(a.status, DL_ERR_CAPACITY, I.b);
      }
    }
    if (item + GW < total) { load_item(item + GW, NI); prefetch(NI); }

    float m_run = -INFINITY, l_run = 0.f;          // l_run: this lane's share of the sum
    float acc[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

    for (int st = 0; st < I.nst; ++st, ++consumed) {
      const int slot = consumed % NS;
      mbar_wait(smem_u32(&bars[slot]), (consumed / NS) & 1, abort_flag);
      const int nr = min(RS, I.rows - st * RS);
      if (nr > 0) {
        const uint32_t tile = smem_u32(my_tiles + (size_t)slot * kMmaStage);
        if (nr < RS) {
          // ragged last tile: rows >= nr hold unrelated data; zero them in V so that 0 * x stays 0
          char* vz = my_tiles + (size_t)slot * kMmaStage + 2 * kMmaBox;
          for (int u = lane; u < 2 * RS * 8; u += 32) {
            const int r = (u >> 3) & (RS - 1);
            if (r >= nr) *reinterpret_cast<uint4*>(vz + (u >> 7) * kMmaBox + r * 128 + (u & 7) * 16) = make_uint4(0, 0, 0, 0);
          }
          __syncwarp();
        }
        // ---- S = q . K^T for 16 rows: two 8-row blocks
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const int chunk = 2 * ks + k_csel;                         // 16-byte chunk of the 256-byte row
          const uint32_t addr = tile + (chunk >> 3) * kMmaBox + k_row * 128 + (((chunk & 7) ^ (k_row & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_16816(s0, qa[2 * ks], qa[2 * ks + 1], b0, b1);
          mma_16816(s1, qa[2 * ks], qa[2 * ks + 1], b2, b3);
        }
        // ---- online softmax; lanes 0-3 hold rows 2t, 2t+1 (block 0) and 8+2t, 9+2t (block 1)
        float sv[4];
        sv[0] = (row0_lane && 2 * t4 < nr) ? s0[0] * a.scale_log2 : -INFINITY;
        sv[1] = (row0_lane && 2 * t4 + 1 < nr) ? s0[1] * a.scale_log2 : -INFINITY;
        sv[2] = (row0_lane && 8 + 2 * t4 < nr) ? s1[0] * a.scale_log2 : -INFINITY;
        sv[3] = (row0_lane && 9 + 2 * t4 < nr) ? s1[1] * a.scale_log2 : -INFINITY;
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        mx = __shfl_sync(0xffffffffu, mx, 0);
        if (mx > m_run) {                                            // warp-uniform
          const float corr = exp2f(m_run - mx);
          l_run *= corr;
#pragma unroll
          for (int i = 0; i < 16; ++i) { acc[i][0] *= corr; acc[i][1] *= corr; }
          m_run = mx;
        }
        const float p0 = exp2f(sv[0] - m_run), p1 = exp2f(sv[1] - m_run);
        const float p2 = exp2f(sv[2] - m_run), p3 = exp2f(sv[3] - m_run);
        l_run += (p0 + p1) + (p2 + p3);
        const uint32_t pa0 = pack_bf16x2(p0, p1), pa2 = pack_bf16x2(p2, p3);
        // ---- O += P . V : 16 blocks of 8 dims
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
          const int chunk = 2 * dp + v_csel;
          const uint32_t addr = tile + (2 + (chunk >> 3)) * kMmaBox + v_row * 128 + (((chunk & 7) ^ (v_row & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(addr, b0, b1, b2, b3);
          mma_16816(acc[2 * dp], pa0, pa2, b0, b1);
          mma_16816(acc[2 * dp + 1], pa0, pa2, b2, b3);
        }
        if (nr < RS) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      __syncwarp();
      if (p_valid && !*abort_flag) {
        if (lane == 0) issue(PI, p_st, slot);
        advance_producer();
      }
    }

    // ---- finish the item: lanes 0-3 own the output (block i: dims 8i + 2t, 8i + 2t + 1)
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    l_run = __shfl_sync(0xffffffffu, l_run, 0);
    uint32_t* outw = reinterpret_cast<uint32_t*>((char*)a.out + bh * RB);
    // the current token's value in the output layout: word 4i + t holds dims 8i + 2t, 8i + 2t + 1
    const uint32_t* vtw = reinterpret_cast<const uint32_t*>((const char*)a.v_t + bh * RB);
    if (I.nch == 1) {
      const float M2 = fmaxf(m_run, s_e);
      const float wc = (m_run == -INFINITY) ? 0.f : exp2f(m_run - M2);
      const float we = exp2f(s_e - M2);
      const float inv = 1.f / (l_run * wc + we);
      if (row0_lane && DL_IN_BOUNDS(a.status, KID_DECODE_MMA, bh * RB + RB - 1, (size_t)a.B * a.H * RB)) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t vw = __ldg(vtw + i * 4 + t4);
          outw[i * 4 + t4] = pack_bf16x2((acc[i][0] * wc + we * bf16lo(vw)) * inv,
                                         (acc[i][1] * wc + we * bf16hi(vw)) * inv);
        }
      }
      continue;
    }
    float* part = a.partial + (bh * a.slots + I.c) * (size_t)(D + 2);
    if (row0_lane && DL_IN_BOUNDS(a.status, KID_DECODE_MMA, (bh * a.slots + I.c) * (size_t)(D + 2) + D + 1,
                                  (size_t)a.B * a.H * a.slots * (D + 2))) {
#pragma unroll
      for (int i = 0; i < 16; ++i) *reinterpret_cast<float2*>(part + i * 8 + 2 * t4) = make_float2(acc[i][0], acc[i][1]);
    }
    if (lane == 0) { part[D] = m_run; part[D + 1] = l_run; }
    __threadfence();
    __syncwarp();
    int ticket = 0;
    if (lane == 0) ticket = atomicAdd(&a.ticket[bh], 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket == I.nch - 1) {
      __threadfence();
      const float* p0 = a.partial + bh * a.slots * (size_t)(D + 2);
      float Mg = s_e;
      for (int cc = 0; cc < I.nch; ++cc) Mg = fmaxf(Mg, __ldcg(p0 + (size_t)cc * (D + 2) + D));
      const float we = exp2f(s_e - Mg);
      float den = we;
      float num[32];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint32_t vw = row0_lane ? __ldg(vtw + i * 4 + t4) : 0u;
        num[2 * i] = we * bf16lo(vw);
        num[2 * i + 1] = we * bf16hi(vw);
      }
      for (int cc = 0; cc < I.nch; ++cc) {
        const float* pc = p0 + (size_t)cc * (D + 2);
        const float mc = __ldcg(pc + D);
        const float wt = (mc == -INFINITY) ? 0.f : exp2f(mc - Mg);
        den = fmaf(__ldcg(pc + D + 1), wt, den);
        if (row0_lane) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float2 v2 = __ldcg(reinterpret_cast<const float2*>(pc + i * 8 + 2 * t4));
            num[2 * i] = fmaf(v2.x, wt, num[2 * i]);
            num[2 * i + 1] = fmaf(v2.y, wt, num[2 * i + 1]);
          }
        }
      }
      const float inv = 1.f / den;
      if (row0_lane) {
#pragma unroll
        for (int i = 0; i < 16; ++i) outw[i * 4 + t4] = pack_bf16x2(num[2 * i] * inv, num[2 * i + 1] * inv);
      }
      if (lane == 0) a.ticket[bh] = 0;
    }
  }

  // A kernel that was allowed to start early must not finish before its predecessor has: whatever
  // follows in the stream (the length commit) relies on all earlier layers being done.
  if (a.overlap) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (*abort_flag) {
    if (lane == 0) {
      report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
      for (int j = max(0, issued - NS); j < issued; ++j)
        for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&bars[j % NS]), (j / NS) & 1); ++i) __nanosleep(40);
    }
  }
  decode_commit(a);
}

// Tensor maps over a cache viewed as [B*H*cap rows][128 dims]: box 64 dims x 16 rows, 128-byte swizzle.
static bool encode_cache_map(void* fn, void* out, const void* base, long long rows) {
  const uint64_t dims[2] = {128ull, (uint64_t)rows};
  const uint64_t strides[1] = {256ull};
  const uint32_t box[2] = {64u, (uint32_t)kMmaRows};
  return encode_bf16_map(fn, reinterpret_cast<CUtensorMap*>(out), base, 2, dims, strides, box);
}

// Encoding a tensor map costs a few microseconds on the host; the same cache tensors come back
// every decode step, so the context remembers the maps it has built (keyed by base and row count).
static bool cached_cache_map(const dl_ctx* ctx, void* out, const void* base, long long rows) {
  for (int i = 0; i < dl_ctx::kMapCache; ++i) {
    const dl_ctx::MapEntry& e = ctx->map_cache[i];
    if (e.base == base && e.rows == rows) { memcpy(out, e.map, 128); return true; }
  }
  dl_ctx::MapEntry& e = ctx->map_cache[ctx->map_next];
  alignas(64) unsigned char tmp[128];
  if (!encode_cache_map(ctx->tmap_encode, tmp, base, rows)) return false;
  memcpy(e.map, tmp, 128);
  e.base = base; e.rows = rows;
  ctx->map_next = (ctx->map_next + 1) % dl_ctx::kMapCache;
  memcpy(out, tmp, 128);
  return true;
}

static cudaError_t launch_mma(const dl_ctx* ctx, DecodeArgs& a, cudaStream_t s) {
  TmapPair maps;
  const long long rows = (long long)a.B * a.H * a.cap;
  if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
  if (!cached_cache_map(ctx, maps.k, a.k_cache, rows) || !cached_cache_map(ctx, maps.v, a.v_cache, rows))
    return cudaErrorInvalidValue;
  const size_t fixed = (size_t)(a.B + 1) * sizeof(int) + 1024 /*alignment*/ + 256;
  const int per_cta = (ctx->smem_optin + 1024) / kMmaCtas - 1024;        // shared memory one CTA may take
  int ns = (int)((per_cta - 256 - (int)fixed) / (kMmaWarps * (kMmaStage + 8)));
  ns = min(ns, 6);
  if (ns < 2) return cudaErrorInvalidConfiguration;
  a.n_stages = ns;
  const size_t smem = (size_t)kMmaWarps * ns * (kMmaStage + 8) + fixed;
  static int attr_set[64];
  int& attr_set_for = attr_set[ctx->device & 63];
  if (attr_set_for != (int)smem) {
    cudaError_t e = cudaFuncSetAttribute(attn_decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set_for = (int)smem;
  }
  // The one-slot mode of a layer stack counts on exactly kMmaCtas CTAs of this kernel fitting an SM (that
  // bounds how many layers can be in flight, hence how many scratch sets are needed): checked once per
  // device and shared-memory size; otherwise a launch takes all slots and overlaps only when unsplit.
  static int occ_for[64], occ_val[64];
  if (occ_for[ctx->device & 63] != (int)smem) {
    int nb = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, attn_decode_mma_kernel, kMmaWarps * 32, smem);
    if (e != cudaSuccess) return e;
    occ_val[ctx->device & 63] = nb;
    occ_for[ctx->device & 63] = (int)smem;
  }
  if (a.one_slot && occ_val[ctx->device & 63] != kMmaCtas) {
    a.one_slot = 0;
    a.overlap = (a.overlap && max_chunks(a) == 1) ? 1 : 0;
  }
  const long long max_items = (long long)a.B * a.H * max_chunks(a);
  const int grid = (int)max(1LL, min((long long)ctx->sm_count * (a.one_slot ? 1 : kMmaCtas), max_items));
  if (!a.overlap) {
    attn_decode_mma_kernel<<<grid, kMmaWarps * 32, smem, s>>>(maps, a);
    return cudaGetLastError();
  }
  // Programmatic stream serialisation: this launch may begin while the previous kernel of the stream
  // (the decode attention of the previous layer, which touches other caches and outputs) drains.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kMmaWarps * 32); cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attn_decode_mma_kernel, maps, a);
}

template <typename T, int D>
static cudaError_t launch_t(const dl_ctx* ctx, DecodeArgs& a, cudaStream_t s) {
  constexpr int RB = D * (int)sizeof(T);
  if (sizeof(T) == 2 && D == 128 && ctx->tmap_encode != nullptr && ctx->opt.decode_impl != 1)
    return launch_mma(ctx, a, s);
  // 4 KB of K+V per stage and 16 warps: 3 stages per warp, 192 KB in flight per SM
  constexpr int RS = (RB >= 512) ? 4 : (RB == 256 ? 8 : 16);
  return launch_cfg<T, D, RS, 16>(ctx, a, s);
}

// Host side of decode_chunks(): the explicit chunk (0 = none) and the number of items per (b, h).
static void pick_split(const dl_ctx* ctx, DecodeArgs& a) {
  a.chunk = 0;
  if (ctx->opt.decode_chunk > 0)
    a.chunk = max(kDecodeMinChunk, (ctx->opt.decode_chunk + kDecodeRowAlign - 1) / kDecodeRowAlign * kDecodeRowAlign);
  const bool mma = ctx->desc.dtype == DL_BF16 && ctx->desc.head_dim == 128 && ctx->tmap_encode && ctx->opt.decode_impl != 1;
  const long long warps = (long long)ctx->sm_count * (mma ? 8 : 16);
  a.per_bh = (int)max(1LL, warps / ((long long)a.B * a.H));
}
static int scratch_slots(const DecodeArgs& a) { return max_chunks(a) + 1; }

cudaError_t launch_attn_decode(const dl_ctx* ctx, const void* q, const void* k_t, const void* v_t,
                               void* k_cache, void* v_cache, const int32_t* cache_len,
                               const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                               bool overlap_prev, int scratch_set, cudaStream_t s, int32_t* commit_len,
                               int commit_slot) {
  if (B == 0) return cudaSuccess;
  if (B > kMaxDecodeBatch) return cudaErrorInvalidValue;
  const dl_model_desc& d = ctx->desc;
  DecodeArgs a;
  a.commit_len = keep ? commit_len : nullptr;
  a.commit_count = ctx->ws.dec_commit + (commit_slot & 1);
  a.q = q; a.k_t = k_t; a.v_t = v_t; a.k_cache = k_cache; a.v_cache = v_cache;
  a.cache_len = cache_len; a.keep = keep; a.out = out;
  a.status = ctx->ws.status;
  a.B = B; a.H = d.n_heads; a.cap = cap;
  pick_split(ctx, a);
  a.slots = ctx->ws.dec_slots;
  // the scratch of split sequences: one of three sets, so that launches in flight together differ
  const size_t set = (size_t)(scratch_set % kDecodeScratchSets);
  a.ticket = ctx->ws.dec_ticket + set * (size_t)ctx->ws.max_batch * d.n_heads;
  a.partial = ctx->ws.dec_partial + set * (size_t)ctx->ws.max_batch * d.n_heads * ctx->ws.dec_slots * (d.head_dim + 2);
  // Inside a layer stack a launch takes ONE CTA slot per SM (where the GPU has two): the next layer's
  // launch, which may start as soon as this one has, takes the other, so two layers stream side by side
  // and a layer's start-up and tail are covered by its neighbour's traffic.  How many layers can be in
  // flight: a CTA of layer l+1 stays until layer l has completed (its grid-dependency wait), so the
  // first sm_count CTAs to leave are layer l's; layer l+2 has started everywhere only once they have
  // left, and layer l+3 cannot start before that.  So at most layers l, l+1, l+2 overlap: three scratch sets.
  // Outside a stack, or with fewer items than SMs, a launch uses both slots and overlaps its predecessor
  // only if it needs no scratch.
  const bool mma_path = d.dtype == DL_BF16 && d.head_dim == 128 && ctx->tmap_encode && ctx->opt.decode_impl != 1;
  a.one_slot = (mma_path && ctx->opt.in_layer_stack && (long long)B * d.n_heads * max_chunks(a) >= ctx->sm_count) ? 1 : 0;
  a.overlap = (overlap_prev && (max_chunks(a) == 1 || a.one_slot)) ? 1 : 0;
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
  DecodeArgs a;
  a.B = B; a.H = d.n_heads; a.cap = cap;
  a.commit_len = nullptr; a.commit_count = nullptr;
  pick_split(ctx, a);
  a.overlap = 0;
  a.one_slot = 0;
  const int slots = scratch_slots(a);
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
    a.q = q_t; a.k_t = k_t; a.v_t = v_t; a.k_cache = k_cache; a.v_cache = v_cache;
    a.cache_len = cache_len; a.keep = keep; a.out = out;
    a.ticket = static_cast<int32_t*>(base);
    a.partial = reinterpret_cast<float*>(static_cast<char*>(base) + ticket_bytes);
    a.status = ctx->ws.base ? ctx->ws.status : nullptr;
    a.slots = slots; a.n_stages = 0;
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
