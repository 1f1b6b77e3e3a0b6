// Definitions shared by the tensor-core prefill attention kernels: tile constants, small arithmetic
// wrappers, tensor maps, the work-item walker and the register-budget instructions.
#pragma once

#include "common.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kAtBM = 128, kAtBN = 128, kAtThreads = 384;
constexpr int kAtTile = 2 * 128 * 128;                // 32 KB: two [128 rows][64 dims] halves
constexpr int kAtOffBar = 7 * kAtTile;                // seven tiles (see attn_prefill_tc.cu), then the barriers
constexpr size_t kAtSmem = kAtOffBar + 512;           // 229888 bytes: one CTA per SM
constexpr uint32_t kAtColO = 0, kAtColS = 128, kAtLaneCols = 256;   // tensor-memory columns of one lane: O | S
constexpr float kRescaleStep = 8.0f;                  // log2 units by which the maximum may lag
constexpr int kAtTopRows = 16;                        // a top tile of at most this many rows is left to at_top_rows()

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

// Tensor maps: Q, K and V each with boxes of 128, 64, 32 and 16 rows (index 0..3), so that a ragged
// tile at the end of a sequence is fetched with the smallest box that covers it; O for the stores.
struct AtMaps {
  alignas(64) unsigned char q[4][128]; alignas(64) unsigned char k[4][128];
  alignas(64) unsigned char v[4][128]; alignas(64) unsigned char o[128];
};
// index of the smallest box (128 >> index rows) that covers `rows` (a multiple of 16 in 16..128)
__device__ __forceinline__ int at_box(int rows) { return rows > 64 ? 0 : rows > 32 ? 1 : rows > 16 ? 2 : 3; }

struct AtArgs {
  const int32_t* cache_len; __nv_bfloat16* out; DeviceStatus* status;
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;   // the tensors the maps describe
  int32_t B, H, cap, n_max, q_pairs, item_rows;     // item_rows: query rows per work item (256: a pair of tiles; 128)
  float scale_log2;
};

// Work item -> (b, h, pair p of query tiles).  Pair p counts from the sequence's end: it covers rows
// [q_hi - 256, q_hi) with q_hi = n - 256 p, clipped at row 0; its keys are [0, q_hi) in n_kv tiles.
struct AtItem { int b, h, q_hi, n, n_kv, row_base, swap, cut; };   // cut: a tile of at most `cut` rows is nobody's lane

// One lane's share of an item: rows [q0, q_hi) are owned (the Q tile is loaded from row q0, 128 rows;
// a tile clipped at the top of the sequence loads rows [0, 128) and owns the first q_hi of them),
// keys [0, q_hi) in n_tiles tiles.  The later query tile of a pair has one key tile more than the
// earlier one, so the lanes swap tiles from one item to the next (I.swap) and do the same work.
struct AtLane { int q0, q_hi, n_tiles; bool exists; };
__device__ __forceinline__ AtLane at_lane(const AtItem& I, int lane_id) {
  AtLane L;
  L.q_hi = I.q_hi - (lane_id ^ I.swap) * kAtBM;
  L.exists = L.q_hi > I.cut;
  L.q0 = max(L.q_hi - kAtBM, 0);
  L.n_tiles = (L.q_hi + kAtBN - 1) / kAtBN;
  return L;
}
// keys of tile j that a lane's MMAs cover: all 128, or what is left of [0, q_hi) rounded up to 16
__device__ __forceinline__ int at_cols(const AtLane& L, int j) {
  return min(kAtBN, (L.q_hi - j * kAtBN + 15) & ~15);
}

// A load the compiler may not sink towards its use (the point is to have it in flight early).
__device__ __forceinline__ int ld_early(const int32_t* p) {
  int v;
  asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

// Walks the items of this CTA in the order every role uses: item = p * B * H + b * H + h, stepping by the
// grid size, so all pairs 0 (the longest) come first.  The position is kept as (p, b, h) and advanced by
// additions (a division per item and role is what an item's set-up cannot afford); the length of the NEXT
// item's sequence is requested one item early, so its latency never sits in front of a role's first wait.
// (Walking head by head instead, all pairs of a head side by side, halves the DRAM reads on long contexts
// - K and V of a head are then fetched once - but measured 20-60 % slower: the kernel is not DRAM-bound.
// Rounds that run forwards and backwards in turn, to even out the CTAs' totals, measured 7-12 % slower too.)
constexpr bool kAtSwapLanes = true;
struct AtWalker {
  const AtArgs& a;
  int p, b, h, len, db, dh, sw;               // next item, its length (in flight), the step as (db, dh), swap bit
  __device__ __forceinline__ explicit AtWalker(const AtArgs& a_) : a(a_) {
    const int bh_count = a.B * a.H;
    p = (int)blockIdx.x / bh_count;
    const int bh = (int)blockIdx.x - p * bh_count;
    b = bh / a.H;
    h = bh - b * a.H;
    db = (int)gridDim.x / a.H;
    dh = (int)gridDim.x - db * a.H;
    sw = 0;
    len = p < a.q_pairs ? ld_early(a.cache_len + b) : 0;
  }
  // Advances to the next item that exists (a sequence of 256 p rows or fewer has no pair p; with cut > 0 neither
  // has one whose later tile would have at most `cut` rows).
  __device__ __forceinline__ bool next(AtItem& I, int cut) {
    for (;;) {
      if (p >= a.q_pairs) return false;
      const int cp = p, cb = b, ch = h, clen = len;
      h += dh;
      b += db;
      if (h >= a.H) { h -= a.H; ++b; }
      while (b >= a.B) { b -= a.B; ++p; }
      if (p < a.q_pairs) len = ld_early(a.cache_len + b);
      I.b = cb;
      I.h = ch;
      I.n = min(max(clen, 0), min(a.cap, a.n_max));
      I.q_hi = I.n - cp * a.item_rows;
      if (I.q_hi <= cut) continue;
      I.cut = cut;
      I.n_kv = (I.q_hi + kAtBN - 1) / kAtBN;
      I.row_base = (cb * a.H + ch) * a.cap;                         // first row of this (b, h) in the caches
      I.swap = (kAtSwapLanes && a.item_rows == 2 * kAtBM) ? sw : 0;
      sw ^= 1;
      return true;
    }
  }
};

// Register budget per role (the kernel starts every thread at 168): the producer / MMA warps give
// registers back, the softmax warps take them to hold a whole score row.
constexpr int kAtRegsSmall = 72, kAtRegsSoftmax = 216;
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// Host side, shared by the launchers: the tensor maps of one call and the kernel's arguments.
inline cudaError_t at_prepare(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max, float scale, void* out,
                              AtMaps* maps, AtArgs* a, long long* items) {
  const dl_model_desc& d = ctx->desc;
  const long long rows = (long long)B * d.n_heads * cap;
  if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
  const uint64_t dims[2] = {128ull, (uint64_t)rows};
  const uint64_t strides[1] = {256ull};
  // out [B][n_max][H][128]: 32 rows x 32 columns of one head per store
  const uint64_t dims_o[4] = {128ull, (uint64_t)d.n_heads, (uint64_t)n_max, (uint64_t)B};
  const uint64_t strides_o[3] = {256ull, 256ull * d.n_heads, 256ull * d.n_heads * n_max};
  const uint32_t box_o[4] = {32u, 1u, 32u, 1u};
  for (int i = 0; i < 4; ++i) {
    const uint32_t box[2] = {64u, 128u >> i};
    if (!encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps->q[i]), q, 2, dims, strides, box) ||
        !encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps->k[i]), k_cache, 2, dims, strides, box) ||
        !encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps->v[i]), v_cache, 2, dims, strides, box))
      return cudaErrorInvalidValue;
  }
  if (!encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps->o), out, 4, dims_o, strides_o, box_o,
                       CU_TENSOR_MAP_SWIZZLE_64B))
    return cudaErrorInvalidValue;
  a->cache_len = cache_len; a->out = static_cast<__nv_bfloat16*>(out); a->status = ctx->ws.base ? ctx->ws.status : nullptr;
  a->q = static_cast<const __nv_bfloat16*>(q); a->k = static_cast<const __nv_bfloat16*>(k_cache);
  a->v = static_cast<const __nv_bfloat16*>(v_cache);
  a->item_rows = 2 * kAtBM;
  a->B = B; a->H = d.n_heads; a->cap = cap; a->n_max = n_max; a->q_pairs = (n_max + a->item_rows - 1) / a->item_rows;
  a->scale_log2 = scale * 1.4426950408889634f;
  *items = (long long)B * d.n_heads * a->q_pairs;
  return *items >= (1LL << 31) ? cudaErrorInvalidValue : cudaSuccess;
}

}  // namespace dl
