// The few rows at the top of a sequence (Eq. 1 on rows 0 .. s-1, s <= 16, which attend keys 0 .. s-1 only).
// With query tiles aligned to the end of a sequence, a length of 128 m + r with r <= 16 leaves a top tile of r
// rows: as a work item of the tensor-memory pipeline it would cost a whole item's hand-overs for a 16 x 16 block of
// scores.  One otherwise idle warp computes it instead, with warp-level MMAs on operands loaded straight from
// global memory (12 KB in all), beside the pipeline and off its K/V ring.
#pragma once

#include "attn_prefill.cuh"
#include "attn_prefill_softmax.cuh"

namespace dl {

__device__ __forceinline__ void mma_bf16_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Rows [0, s) of sequence (I.b, I.h), s in 1..16.  Called by all 32 lanes of one warp.
// Fragment layout of m16n8k16 (g = lane / 4, t = lane % 4): A holds rows g and g + 8, columns 2t, 2t+1 and
// 2t+8, 2t+9; B holds row (of the transposed operand) g, the same columns; C rows g and g + 8, columns 2t, 2t+1.
static __device__ __forceinline__ void at_top_rows(const AtArgs& a, const AtItem& I, int s, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const __nv_bfloat16* qb = a.q + (size_t)I.row_base * 128;
  const __nv_bfloat16* kb = a.k + (size_t)I.row_base * 128;
  const __nv_bfloat16* vb = a.v + (size_t)I.row_base * 128;
  auto pair_of = [&](const __nv_bfloat16* base, int row, int d) -> uint32_t {       // two dims of one row, 0 past row s
    return row < s ? __ldg(reinterpret_cast<const uint32_t*>(base + (size_t)row * 128 + d)) : 0u;
  };
  // ---- S = Q K^T: 16 rows x 16 keys (two blocks of 8 keys)
  float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll 1
  for (int ks = 0; ks < 8; ++ks) {
    const int d0 = ks * 16 + 2 * t;
    const uint32_t a0 = pair_of(qb, g, d0), a1 = pair_of(qb, g + 8, d0);
    const uint32_t a2 = pair_of(qb, g, d0 + 8), a3 = pair_of(qb, g + 8, d0 + 8);
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
      mma_bf16_16816(c[nb], a0, a1, a2, a3, pair_of(kb, nb * 8 + g, d0), pair_of(kb, nb * 8 + g, d0 + 8));
  }
  // ---- softmax of rows g and g + 8 (a row's 16 scores sit in the four lanes of its group): key <= row only
  uint32_t pa[4];
  float inv[2];
#pragma unroll
  for (int hf = 0; hf < 2; ++hf) {
    const int r = g + 8 * hf;
    float v[4];
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int key = nb * 8 + 2 * t + j;
        v[nb * 2 + j] = (key <= r && r < s) ? c[nb][2 * hf + j] * a.scale_log2 : -INFINITY;
      }
    float m = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
    float e[4], sum = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) { e[i] = (v[i] == -INFINITY) ? 0.f : fast_exp2(v[i] - m); sum += e[i]; }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    inv[hf] = sum > 0.f ? 1.0f / sum : 0.f;
    pa[hf] = cvt_bf16x2(e[0], e[1]);            // keys 2t, 2t+1     (A columns 2t..)
    pa[2 + hf] = cvt_bf16x2(e[2], e[3]);        // keys 2t+8, 2t+9   (A columns 2t+8..)
  }
  // ---- O = P V, 32 dims at a time; V rows past s count as zero (their P is zero, and 0 * x must stay 0)
  auto v_pair = [&](int key, int dim) -> uint32_t {                                 // V[key][dim], V[key+1][dim]
    const uint32_t lo = key < s ? __ldg(reinterpret_cast<const unsigned short*>(vb + (size_t)key * 128 + dim)) : 0u;
    const uint32_t hi = key + 1 < s ? __ldg(reinterpret_cast<const unsigned short*>(vb + (size_t)(key + 1) * 128 + dim)) : 0u;
    return lo | (hi << 16);
  };
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    float o[4][4];
#pragma unroll
    for (int nb = 0; nb < 4; ++nb) {
      o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
      const int dim = pass * 32 + nb * 8 + g;
      mma_bf16_16816(o[nb], pa[0], pa[1], pa[2], pa[3], v_pair(2 * t, dim), v_pair(2 * t + 8, dim));
    }
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int r = g + 8 * hf;
      if (r >= s) continue;
      if (!DL_IN_BOUNDS(a.status, KID_PREFILL_TOP, (((size_t)I.b * a.n_max + r) * a.H + I.h) * 128 + 127,
                        (size_t)a.B * a.n_max * a.H * 128))
        continue;
      uint32_t* orow = reinterpret_cast<uint32_t*>(a.out + (((size_t)I.b * a.n_max + r) * a.H + I.h) * 128 + pass * 32 + 2 * t);
#pragma unroll
      for (int nb = 0; nb < 4; ++nb) orow[nb * 4] = cvt_bf16x2(o[nb][2 * hf] * inv[hf], o[nb][2 * hf + 1] * inv[hf]);
    }
  }
}

}  // namespace dl
