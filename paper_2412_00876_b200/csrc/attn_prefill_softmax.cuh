// The softmax of a score tile in the tensor-core prefill attention kernel (attn_prefill_tc.cu) and its arithmetic helpers.
#pragma once

#include "attn_prefill.cuh"

namespace dl {

__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// 2^x for two values x <= 0 on the FMA pipe: x = i + f with i integral and f in [-0.5, 0.5] (the rounding
// of x + 1.5 * 2^23), a cubic for 2^f (relative error 7.5e-5, far below the bf16 rounding of P) and i added
// to the exponent bits.  Inputs below -126 (masked scores are -inf) give at most 2^-126.
__device__ __forceinline__ void poly_exp2_x2(uint64_t x2, float& o0, float& o1) {
  const float magic = 12582912.f;
  float x0, x1;
  unpack2(x2, x0, x1);
  x0 = fmaxf(x0, -126.f);
  x1 = fmaxf(x1, -126.f);
  const uint64_t xc = pack2(x0, x1);
  const uint64_t t = fadd2(xc, pack2(magic, magic));
  const uint64_t fi = fadd2(t, pack2(-magic, -magic));
  const uint64_t f = ffma2(fi, pack2(-1.f, -1.f), xc);
  uint64_t p = ffma2(pack2(0.0551716611f, 0.0551716611f), f, pack2(0.242611125f, 0.242611125f));
  p = ffma2(p, f, pack2(0.693260968f, 0.693260968f));
  p = ffma2(p, f, pack2(0.999928057f, 0.999928057f));
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(t, t0, t1);
  o0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(t0) << 23));
  o1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(t1) << 23));
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}

// The rare path of the softmax below: the row's maximum in use has been raised, so everything the row has
// accumulated under the old one is multiplied by corr = 2^(old - new): its 128 columns of O in tensor memory
// (if the item has accumulated anything yet) and the n_stored chunks of P (16 columns of bf16 pairs each) that
// this tile has already written.  Kept out of line: it runs once or twice per row, not once per tile.
static __device__ __noinline__ void at_rescale_row(uint32_t o_addr, uint32_t p_addr, int n_stored, float corr, int o_valid) {
  const uint64_t corr2 = pack2(corr, corr);
  if (o_valid) {
#pragma unroll 1
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t o[32];
      tmem_ld32(o_addr + cc * 32, o);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        float y0, y1;
        unpack2(fmul2(pack2(__uint_as_float(o[i]), __uint_as_float(o[i + 1])), corr2), y0, y1);
        o[i] = __float_as_uint(y0);
        o[i + 1] = __float_as_uint(y1);
      }
      tmem_st32(o_addr + cc * 32, o);
    }
  }
#pragma unroll 1
  for (int cc = 0; cc < n_stored; ++cc) {
    uint32_t w[16];
    tmem_ld16(p_addr + cc * 16, w);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = cvt_bf16x2(bf16lo(w[i]) * corr, bf16hi(w[i]) * corr);
    tmem_st16(p_addr + cc * 16, w);
  }
  tmem_st_wait();
}

__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr) : "memory");
}

// Softmax of one 128 x 128 score tile, one query row per thread, in four steps of 32 columns: P = 2^(S * scale_log2
// - m_used) goes, as bf16 pairs, over the first 64 columns of the score buffer (step by step: the scores it
// overwrites are in registers by then) and the row sum is added to l_run.  The maximum in use lags: a step whose
// own maximum is more than 2^8 above it raises it first (rescaling what the row holds so far, see at_rescale_row),
// so that no exponential exceeds 2^8; a row's first step sets it.  Per step: mask (only where the chunk reaches
// past the warp's first row), maximum, all multiply-adds, then the registers of the raw scores take the next
// chunk's load while the exponentials run (NPOLY of every four pairs as a cubic on the FMA pipe, the rest on the
// special-function unit), row sums, packing, store.
// The loop is NOT unrolled, and its body is kept small: a warp is bound by instruction fetch once the body of a
// tile outgrows its scheduler's instruction cache, which it shares with the other lane's warp of the same
// quadrant.  Fully unrolled (4 chunks) the pass cost 15 % of the kernel's time more than in two rolled halves of 64
// columns, and those 3 % more than this form on short contexts.
//   n_ch: 32-column chunks that some row of the warp may see (chunks beyond get P = 0); column c is visible to this
//   row iff c <= vis; owned: the row belongs to this tile; o_valid: the item has accumulated into O already.
template <int NPOLY>
__device__ __forceinline__ void at_softmax_chunks(uint32_t s_addr, uint32_t o_addr, int n_ch, int vis, int c0_minus_r0,
                                                  bool owned, int o_valid, float scale_log2, float& m_used, float& l_run) {
  const int n_q = max(min(4, n_ch), 0);
  const uint64_t sc2 = pack2(scale_log2, scale_log2);
  uint32_t buf[32];
  uint64_t l2[4] = {0ull, 0ull, 0ull, 0ull};
  if (n_q > 0) {
    tmem_ld32(s_addr, buf);
    tmem_ld_wait();
  }
#pragma unroll 1
  for (int q = 0; q < n_q; ++q) {
    if (c0_minus_r0 + 32 * q + 31 > 0) {                         // the chunk reaches past the warp's first row
      const int v = vis - 32 * q;
#pragma unroll
      for (int c = 0; c < 32; ++c)
        if (c > v) buf[c] = 0xFF800000u;                         // -inf
    }
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
        mx4[w] = fmax3(mx4[w], __uint_as_float(buf[c + 2 * w]), __uint_as_float(buf[c + 2 * w + 1]));
    }
    const float mc = fmax3(mx4[0], mx4[1], fmaxf(mx4[2], mx4[3])) * scale_log2;
    const bool need = owned && mc > m_used + kRescaleStep;
    if (__any_sync(0xffffffffu, need)) {
      const float corr = need ? fast_exp2(m_used - mc) : 1.0f;   // an unset maximum (-inf) gives 0
      if (need) m_used = mc;
      l_run *= corr;
      const uint64_t corr2 = pack2(corr, corr);
#pragma unroll
      for (int i = 0; i < 4; ++i) l2[i] = fmul2(l2[i], corr2);
      at_rescale_row(o_addr, s_addr, q, corr, o_valid);
    }
    const uint64_t nm2 = pack2(-m_used, -m_used);
    uint64_t t[16];
#pragma unroll
    for (int c = 0; c < 16; ++c)
      t[c] = ffma2(pack2(__uint_as_float(buf[2 * c]), __uint_as_float(buf[2 * c + 1])), sc2, nm2);
    if (q + 1 < n_q) tmem_ld32(s_addr + 32 * (q + 1), buf);      // the raw scores are used up: next chunk into their registers
    uint32_t pk[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      float e0, e1;
      if ((c & 3) < NPOLY) {
        poly_exp2_x2(t[c], e0, e1);
      } else {
        unpack2(t[c], e0, e1);
        e0 = fast_exp2(e0);
        e1 = fast_exp2(e1);
      }
      l2[c & 3] = fadd2(l2[c & 3], pack2(e0, e1));
      pk[c] = cvt_bf16x2(e0, e1);
    }
    tmem_st16(s_addr + 16 * q, pk);
    tmem_ld_wait();
  }
  if (n_q < 4) {
    uint32_t z[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll 1
    for (int q = n_q; q < 4; ++q) tmem_st16(s_addr + 16 * q, z);
  }
  float la, lb;
  unpack2(fadd2(fadd2(l2[0], l2[1]), fadd2(l2[2], l2[3])), la, lb);
  l_run += la + lb;
  tmem_st_wait();
}

}  // namespace dl
