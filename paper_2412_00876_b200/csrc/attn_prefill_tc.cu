// Prefill attention over the reduced set on the tensor cores (Eq. 1 applied to S^{P*}):
// row i of a sequence's compact context attends rows 0..i of the same context.
// bf16, head_dim 128.  Persistent CTAs, two per SM (one CTA's softmax overlaps the other's MMAs),
// walk work items (sequence, head, 128-row query tile), longest tiles first; tensor memory, barriers
// and the pipelines live across items, so an item's loads start while the previous one finishes.
// Query tiles are aligned to the END of a sequence (rows [n-128(t+1), n-128t)), so the ragged tile is
// the one at the top of the causal triangle, where it needs the fewest key tiles.
//   warp 0    : TMA producer.  Q of an item (two 64-dim halves) as soon as the previous item's last
//               Q K^T has read the Q buffer; 64-row K tiles and V tiles through two separate 2-slot
//               rings (a K slot is free once its Q K^T has run, long before the V slot of the same
//               tile, so the next K is in flight a whole softmax earlier), all with the 128-byte swizzle;
//   warp 1    : tensor-memory allocation and the single MMA-issuing thread:
//               S = Q K^T (128 x 64, K-major operands from shared memory) into one of two S buffers,
//               O += P V (P read from tensor memory, V as an MN-major shared-memory operand);
//               the next tile's Q K^T is issued before this tile's P V so it runs during the softmax;
//   warps 2-5 : softmax, one query row per thread, straight out of tensor memory.  The running
//               maximum is only raised when it grows by more than 2^8 (then O is rescaled in tensor
//               memory), so most tiles never touch O.  P (bf16) overwrites the first half of its
//               own S buffer.  The same warps normalise O and store the output rows, staged
//               through a small per-warp buffer so that each store instruction writes whole
//               64-byte row segments.
// Tensor memory: O 128 columns, S0 and S1 64 columns each (256 columns per CTA, 512 per SM).
// Barrier phases are driven by running counters (tiles, K/V stages, items) that every role advances
// identically.  Rows past a sequence's length are fetched with the tile (they are masked); in the
// last tile the surplus V rows are zeroed in shared memory first, since 0 * x must stay 0 for any
// bit pattern.  Every wait is bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kAtBM = 128, kAtBN = 64, kAtStages = 2, kAtThreads = 192;
constexpr int kAtQBytes = 2 * kAtBM * 128;            // 32 KB: two [128 rows][64 dims] halves
constexpr int kAtTile = 2 * kAtBN * 128;              // 16 KB: two [64 rows][64 dims] halves
constexpr int kAtStage = 2 * kAtTile;                 // K tile + V tile
constexpr int kAtOutStage = 4 * 2048;                 // per softmax warp: 32 rows x 32 columns of bf16 output
constexpr size_t kAtSmem = kAtQBytes + kAtStages * kAtStage + kAtOutStage + 1024 + 256;
constexpr uint32_t kAtColO = 0, kAtColS = 128;        // tensor-memory columns: O | S0 | S1
constexpr float kRescaleStep = 8.0f;                  // log2 units by which the maximum may lag

// 2^x on the special-function unit (x <= 0 here; -inf gives 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// max of three in one instruction
__device__ __forceinline__ float fmax3(float x, float y, float z) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(x), "f"(y), "f"(z));
  return r;
}

// two fp32 lanes in one 64-bit register: fused multiply-add and add on both at once
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t x, uint64_t y, uint64_t z) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(x), "l"(y), "l"(z));
  return r;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t x, uint64_t y) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(x), "l"(y));
  return r;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t x, uint64_t y) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(x), "l"(y));
  return r;
}

struct AtMaps { alignas(64) unsigned char q[128]; alignas(64) unsigned char k[128]; alignas(64) unsigned char v[128]; };

struct AtArgs {
  const int32_t* cache_len; __nv_bfloat16* out; DeviceStatus* status;
  int32_t B, H, cap, n_max, q_tiles;
  float scale_log2;
};

// Work item -> (b, h, query tile).  Tile t counts from the sequence's end (the longest first): it owns
// rows [q_hi - 128, q_hi) with q_hi = n - 128 t; the tile at the top is clipped to start at row 0 (it
// loads rows [0, 128) and owns the first q_hi of them).  Returns false for a tile the sequence lacks.
struct AtItem { int b, h, q0, q_hi, n, n_tiles, row_base; };
__device__ __forceinline__ bool at_item(const AtArgs& a, int item, AtItem& I) {
  const int bh_count = a.B * a.H;
  const int t = item / bh_count;
  const int bh = item - t * bh_count;
  I.b = bh / a.H;
  I.h = bh - I.b * a.H;
  I.n = min(max(a.cache_len[I.b], 0), min(a.cap, a.n_max));
  I.q_hi = I.n - t * kAtBM;
  if (I.q_hi <= 0) return false;
  I.q0 = max(I.q_hi - kAtBM, 0);
  I.n_tiles = (I.q_hi + kAtBN - 1) / kAtBN;                       // keys any owned row may see: [0, q_hi)
  I.row_base = bh * a.cap;                                        // first row of this (b, h) in the caches
  return true;
}

__global__ void __launch_bounds__(kAtThreads, 2)
attn_prefill_tc_kernel(const __grid_constant__ AtMaps maps, const AtArgs a) {
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  char* q_s = smem;
  char* st_s = smem + kAtQBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(st_s + kAtStages * kAtStage);
  uint64_t* q_full = bars;                 // [1] per item: Q has landed
  // Tile g of a CTA's running count uses slot g & 1 of the K ring, the V ring, the S buffers and of
  // every [2] barrier below, in phase (g >> 1) & 1.  A waiter is never two uses of a slot behind.
  uint64_t* k_full = bars + 1;             // [2] K tile has landed
  uint64_t* v_full = bars + 3;             // [2] V tile has landed
  uint64_t* s_full = bars + 5;             // [2] Q K^T of the tile has completed: S is ready, the K slot is free
  uint64_t* p_full = bars + 7;             // [2] P of the tile is in tensor memory (4 warps)
  uint64_t* pv_done = bars + 9;            // [2] P V of the tile has completed: O is at rest, the V slot is free
  uint64_t* q_empty = bars + 11;           // [1] per item: its last Q K^T has read the Q buffer
  uint64_t* o_free = bars + 12;            // [1] per item: the epilogue has read O (4 warps)
  char* o_stage = st_s + kAtStages * kAtStage + 256;
  __shared__ uint32_t sh_tmem;
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int items = a.B * a.H * a.q_tiles;

  if (tid == 0) {
    sh_abort = 0;
    mbar_init(smem_u32(q_full), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&k_full[i]), 1);
      mbar_init(smem_u32(&v_full[i]), 1);
      mbar_init(smem_u32(&s_full[i]), 1);
      mbar_init(smem_u32(&p_full[i]), 4);
      mbar_init(smem_u32(&pv_done[i]), 1);
    }
    mbar_init(smem_u32(q_empty), 1);
    mbar_init(smem_u32(o_free), 4);
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(&sh_tmem), 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh_tmem;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(maps.q);
      const CUtensorMap* mk = reinterpret_cast<const CUtensorMap*>(maps.k);
      const CUtensorMap* mv = reinterpret_cast<const CUtensorMap*>(maps.v);
      tma_prefetch_desc(mq); tma_prefetch_desc(mk); tma_prefetch_desc(mv);
      int n_item = 0, gk = 0, gv = 0;                                  // items / K tiles / V tiles issued so far
      bool q_pending = false, ok = true;
      // tile g of this CTA's running count -> slot g & 1 of either ring
      // (`freed` completes when the MMAs that read the slot's previous tile have)
      auto load_tile = [&](uint64_t* full, uint64_t* freed, const CUtensorMap* m, int g, int r, int off) {
        const int s = g & 1;
        if (g >= 2 && !mbar_wait(smem_u32(&freed[s]), ((g >> 1) & 1) ^ 1, abort_flag)) return false;
        const uint32_t fb = smem_u32(&full[s]);
        mbar_expect_tx(fb, kAtTile);
        char* st = st_s + (size_t)s * kAtStage + off;
        tma_load_2d(smem_u32(st), m, 0, r, fb);
        tma_load_2d(smem_u32(st + kAtBN * 128), m, 64, r, fb);
        return true;
      };
      for (int item = blockIdx.x; item < items && ok && !*abort_flag; item += gridDim.x) {
        AtItem I;
        if (!at_item(a, item, I)) continue;
        if (!mbar_wait(smem_u32(q_empty), (n_item & 1) ^ 1, abort_flag)) break;
        mbar_expect_tx(smem_u32(q_full), kAtQBytes);
        tma_load_2d(smem_u32(q_s), mq, 0, I.row_base + I.q0, smem_u32(q_full));
        tma_load_2d(smem_u32(q_s + kAtBM * 128), mq, 64, I.row_base + I.q0, smem_u32(q_full));
        q_pending = true;
        ++n_item;
        // same order as the MMA warp consumes them: K(0), then K(j+1) before V(j)
        ok = load_tile(k_full, s_full, mk, gk, I.row_base, 0);
        if (ok) ++gk;
        for (int j = 0; j < I.n_tiles && ok; ++j) {
          if (j + 1 < I.n_tiles) {
            ok = load_tile(k_full, s_full, mk, gk, I.row_base + (j + 1) * kAtBN, 0);
            if (!ok) break;
            ++gk;
          }
          ok = load_tile(v_full, pv_done, mv, gv, I.row_base + j * kAtBN, kAtTile);
          if (ok) ++gv;
        }
      }
      if (*abort_flag) {
        // every copy that was issued must land before the CTA's shared memory is released
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        if (q_pending)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(q_full), (n_item - 1) & 1); ++i) __nanosleep(40);
        for (int j = max(0, gk - 2); j < gk; ++j)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&k_full[j & 1]), (j >> 1) & 1); ++i) __nanosleep(40);
        for (int j = max(0, gv - 2); j < gv; ++j)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&v_full[j & 1]), (j >> 1) & 1); ++i) __nanosleep(40);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16(kAtBM, kAtBN);
      const uint32_t idesc_pv = idesc_bf16(kAtBM, 128, 0, 1);        // B (= V) is MN-major
      const uint64_t q_desc = smem_desc_sw128(smem_u32(q_s));
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(st_s));
      const uint64_t v_desc0 = smem_desc_sw128_mn(smem_u32(st_s) + kAtTile, kAtBN * 128);
      int n_item = 0, g0 = 0;                                          // items / tiles before this item
      for (int item = blockIdx.x; item < items; item += gridDim.x) {
        AtItem I;
        if (!at_item(a, item, I)) continue;
        auto issue_qk = [&](int j) {
          const int g = g0 + j, s = g % kAtStages;
          mbar_wait(smem_u32(&k_full[s]), (g / kAtStages) & 1, abort_flag);
          tc_fence_after();
          const uint64_t kd = k_desc0 + (uint64_t)((s * kAtStage) >> 4);
          const uint32_t d = tmem + kAtColS + (uint32_t)(g & 1) * kAtBN;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_ss(d, q_desc + (uint64_t)(((ks >> 2) * (kAtBM * 128) + (ks & 3) * 32) >> 4),
                   kd + (uint64_t)(((ks >> 2) * (kAtBN * 128) + (ks & 3) * 32) >> 4), idesc_qk, ks != 0);
          mma_commit(smem_u32(&s_full[g & 1]));
          if (j == I.n_tiles - 1) mma_commit(smem_u32(q_empty));       // the Q buffer may be refilled
        };
        mbar_wait(smem_u32(q_full), n_item & 1, abort_flag);
        issue_qk(0);
        for (int j = 0; j < I.n_tiles; ++j) {
          if (j + 1 < I.n_tiles) issue_qk(j + 1);
          const int g = g0 + j, s = g % kAtStages;
          mbar_wait(smem_u32(&p_full[g & 1]), (g >> 1) & 1, abort_flag);
          if (j == 0) mbar_wait(smem_u32(o_free), (n_item & 1) ^ 1, abort_flag);   // previous item's O has been read
          mbar_wait(smem_u32(&v_full[s]), (g / kAtStages) & 1, abort_flag);
          tc_fence_after();
          const uint64_t vd = v_desc0 + (uint64_t)((s * kAtStage) >> 4);
          const uint32_t p_tmem = tmem + kAtColS + (uint32_t)(g & 1) * kAtBN;
#pragma unroll
          for (int ks = 0; ks < kAtBN / 16; ++ks)
            mma_ts(tmem + kAtColO, p_tmem + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), idesc_pv, (j | ks) != 0);
          mma_commit(smem_u32(&pv_done[g & 1]));
        }
        g0 += I.n_tiles;
        ++n_item;
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax / epilogue warps
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                                  // row within the query tile
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    int n_item = 0, g0 = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
      AtItem I;
      if (!at_item(a, item, I)) continue;
      const int grow = I.q0 + row;                                     // row within the sequence
      const int r0 = I.q0 + quad * 32;                                 // this warp's first row
      const int kv_end = I.q_hi;
      float m_used = -INFINITY, l_run = 0.f;
      for (int j = 0; j < I.n_tiles; ++j) {
        const int g = g0 + j, sb = g & 1;
        mbar_wait(smem_u32(&s_full[sb]), (g >> 1) & 1, abort_flag);
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_off + kAtColS + (uint32_t)sb * kAtBN;
        const int c0 = j * kAtBN;
        uint32_t pw[32];
        if (c0 > r0 + 31) {
          // no row of this warp sees a key of this tile: P = 0, nothing else to do
#pragma unroll
          for (int c = 0; c < 32; ++c) pw[c] = 0u;
        } else {
          uint32_t sr[64];
          tmem_ld32(s_addr, sr);
          tmem_ld32(s_addr + 32, sr + 32);
          tmem_ld_wait();
          // raw scores stay unscaled: max commutes with the (positive) scale and the scale is folded into
          // the exponent's FMA.  Only a tile that reaches past the warp's first row needs the causal mask.
          if (c0 + kAtBN - 1 > r0) {
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (c0 + c > grow) sr[c] = 0xFF800000u;                        // -inf
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};     // four independent chains
#pragma unroll
          for (int c = 0; c < 64; c += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
              mx4[u] = fmax3(mx4[u], __uint_as_float(sr[c + 2 * u]), __uint_as_float(sr[c + 2 * u + 1]));
          }
          float mx = fmax3(mx4[0], mx4[1], fmaxf(mx4[2], mx4[3])) * a.scale_log2;
          if (j == 0) {
            m_used = mx;                      // column 0 is visible to every row, so mx is finite
          } else {
            const bool need = mx > m_used + kRescaleStep;
            if (__any_sync(0xffffffffu, need)) {
              // O must be at rest: the P V of the previous tile
              mbar_wait(smem_u32(&pv_done[(g - 1) & 1]), ((g - 1) >> 1) & 1, abort_flag);
              tc_fence_after();
              const float corr = need ? fast_exp2(m_used - mx) : 1.0f;
              if (need) m_used = mx;
              l_run *= corr;
              const uint64_t corr2 = pack2(corr, corr);
#pragma unroll
              for (int cc = 0; cc < 4; ++cc) {
                uint32_t o[32];
                tmem_ld32(tmem + lane_off + kAtColO + cc * 32, o);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                  float x, y;
                  unpack2(fmul2(pack2(__uint_as_float(o[i]), __uint_as_float(o[i + 1])), corr2), x, y);
                  o[i] = __float_as_uint(x);
                  o[i + 1] = __float_as_uint(y);
                }
                tmem_st32(tmem + lane_off + kAtColO + cc * 32, o);
              }
              tmem_st_wait();
            }
          }
          const uint64_t sc2 = pack2(a.scale_log2, a.scale_log2), nm2 = pack2(-m_used, -m_used);
          uint64_t l2[2] = {0ull, 0ull};                                    // two chains of packed row sums
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            float p0, p1;
            unpack2(ffma2(pack2(__uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1])), sc2, nm2), p0, p1);
            p0 = fast_exp2(p0);
            p1 = fast_exp2(p1);
            l2[c & 1] = fadd2(l2[c & 1], pack2(p0, p1));
            __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            pw[c] = *reinterpret_cast<uint32_t*>(&pk);
          }
          float la, lb;
          unpack2(fadd2(l2[0], l2[1]), la, lb);
          l_run += la + lb;
        }
        tmem_st32(s_addr, pw);                                             // P overwrites its own S buffer
        tmem_st_wait();
        if (j == I.n_tiles - 1 && kv_end == I.n && kv_end < c0 + kAtBN) {
          // ragged last tile of the sequence: zero the V rows past its end (both 64-dim halves); past
          // the end of an inner query tile the rows are the sequence's own and P is 0 there
          const int s = g % kAtStages;
          mbar_wait(smem_u32(&v_full[s]), (g / kAtStages) & 1, abort_flag);
          char* vz = st_s + (size_t)s * kAtStage + kAtTile;
          const int first = kv_end - c0;
          for (int u = (warp - 2) * 32 + lane; u < 2 * kAtBN * 8; u += 128) {
            const int r = (u >> 3) & (kAtBN - 1);
            if (r >= first)
              *reinterpret_cast<uint4*>(vz + (u >> 9) * (kAtBN * 128) + r * 128 + (u & 7) * 16) = make_uint4(0, 0, 0, 0);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&p_full[sb]));
      }
      // ---- epilogue: O / l -> bf16 -> out[b][row][h][:], 32 columns at a time through the warp's
      // staging buffer (16-byte units XOR-swizzled by row pair: no bank conflicts either way)
      const int gl = g0 + I.n_tiles - 1;
      mbar_wait(smem_u32(&pv_done[gl & 1]), (gl >> 1) & 1, abort_flag);
      tc_fence_after();
      const float inv = 1.0f / l_run;
      char* so = o_stage + (warp - 2) * 2048;
      __nv_bfloat16* otile = a.out + (((size_t)I.b * a.n_max + I.q0 + quad * 32) * a.H + I.h) * 128;
      const int rows_here = I.q_hi - (I.q0 + quad * 32);               // owned rows among this warp's 32
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t o[32];
        tmem_ld32(tmem + lane_off + kAtColO + cc * 32, o);
        tmem_ld_wait();
        if (cc == 3) {                                   // O is in registers: the next item may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(o_free));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          uint4 w;
          __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(o[8 * u]) * inv, __uint_as_float(o[8 * u + 1]) * inv);
          __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(o[8 * u + 2]) * inv, __uint_as_float(o[8 * u + 3]) * inv);
          __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(o[8 * u + 4]) * inv, __uint_as_float(o[8 * u + 5]) * inv);
          __nv_bfloat162 t3 = __floats2bfloat162_rn(__uint_as_float(o[8 * u + 6]) * inv, __uint_as_float(o[8 * u + 7]) * inv);
          w.x = *reinterpret_cast<uint32_t*>(&t0); w.y = *reinterpret_cast<uint32_t*>(&t1);
          w.z = *reinterpret_cast<uint32_t*>(&t2); w.w = *reinterpret_cast<uint32_t*>(&t3);
          *reinterpret_cast<uint4*>(so + lane * 64 + ((u ^ ((lane >> 1) & 3)) << 4)) = w;
        }
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          const int r = it * 8 + (lane >> 2), u = lane & 3;
          const uint4 w = *reinterpret_cast<const uint4*>(so + r * 64 + ((u ^ ((r >> 1) & 3)) << 4));
          if (r < rows_here) *reinterpret_cast<uint4*>(otile + (size_t)r * a.H * 128 + cc * 32 + u * 8) = w;
        }
        __syncwarp();
      }
      g0 += I.n_tiles;
      ++n_item;
    }
    if (*abort_flag && row == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 256); }
}

bool attn_prefill_tc_supported(const dl_ctx* ctx) {
  const dl_model_desc& d = ctx->desc;
  return d.dtype == DL_BF16 && d.head_dim == 128 && ctx->tmap_encode != nullptr && (size_t)ctx->smem_optin >= kAtSmem;
}

cudaError_t launch_attn_prefill_tc(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max, float scale,
                                   void* out, cudaStream_t s) {
  if (B == 0 || n_max == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  const long long rows = (long long)B * d.n_heads * cap;
  if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
  AtMaps maps;
  const uint64_t dims[2] = {128ull, (uint64_t)rows};
  const uint64_t strides[1] = {256ull};
  const uint32_t box_q[2] = {64u, (uint32_t)kAtBM};
  const uint32_t box_kv[2] = {64u, (uint32_t)kAtBN};
  if (!encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps.q), q, 2, dims, strides, box_q) ||
      !encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps.k), k_cache, 2, dims, strides, box_kv) ||
      !encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps.v), v_cache, 2, dims, strides, box_kv))
    return cudaErrorInvalidValue;
  AtArgs a;
  a.cache_len = cache_len; a.out = static_cast<__nv_bfloat16*>(out); a.status = ctx->ws.base ? ctx->ws.status : nullptr;
  a.B = B; a.H = d.n_heads; a.cap = cap; a.n_max = n_max; a.q_tiles = (n_max + kAtBM - 1) / kAtBM;
  a.scale_log2 = scale * 1.4426950408889634f;
  static int attr_set[64];
  if (!attr_set[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(attn_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmem);
    if (e != cudaSuccess) return e;
    attr_set[ctx->device & 63] = 1;
  }
  const long long items = (long long)B * d.n_heads * a.q_tiles;
  if (items >= (1LL << 31)) return cudaErrorInvalidValue;
  const int grid = (int)std::min<long long>(items, 2LL * ctx->sm_count);
  attn_prefill_tc_kernel<<<grid, kAtThreads, kAtSmem, s>>>(maps, a);
  return cudaGetLastError();
}

}  // namespace dl
