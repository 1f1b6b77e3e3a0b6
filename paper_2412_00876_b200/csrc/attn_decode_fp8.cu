// Decode attention over an 8-bit K/V cache (an extension of Eq. 6; NOT in the paper).
//
// The cache rows are E4M3 bytes (1-4-3, bias 7, largest value 448) with one fp32 scale per head and tensor:
// value = decode(byte) * scale[h].  Decode attention is bound by the bytes it streams, so this halves its floor.
// bf16 models with head_dim 128 only.  Structure as attn_decode_mma_kernel: a persistent grid, a warp per work
// item (sequence, head, chunk of rows), each warp with its own ring of tiles filled by TMA and its own mbarriers;
// here a stage is 32 rows (4 KB of K, 4 KB of V), so the same bytes are in flight.
//   scores:  S = q K^T on mma.sync m16n8k16 with fp16 operands: the bytes go from shared memory to registers with
//            ldmatrix on 16-bit units (two E4M3 values each), every unit becomes an fp16 pair with one conversion
//            (E4M3 is a subset of fp16: exact); the order in which a 16-dim block's dims meet the instruction's
//            k slots is then (4t, 4t+1 | 4t+2, 4t+3) for thread t of a group, and q is laid out to match.
//   values:  O += P V with V read through ldmatrix.trans: a thread gets V[2t][2g, 2g+1] and V[2t+1][2g, 2g+1];
//            a byte permute pairs the two keys of one dim, so a 16-dim chunk is two MMAs, one over its even and one
//            over its odd dims, and thread t ends up with four consecutive dims of the chunk.
//   The scales are applied in fp32 (k_scale with the softmax scale on S, v_scale on the cached part of O).  The
//   current token is attended with its own bf16 k_t, v_t and, if kept, appended as bytes.
#include "common.cuh"
#include "pipeline.cuh"
#include "tc05.cuh"

namespace dl {

constexpr int kF8Warps = 4;                        // warps per CTA
constexpr int kF8Ctas = 2;                         // CTAs per SM
constexpr int kF8Rows = 32;                        // rows per stage
constexpr int kF8Box = kF8Rows * 128;              // one box: 32 rows x 128 bytes
constexpr int kF8Stage = 2 * kF8Box;               // K | V

struct F8Args {
  const void* q; const void* k_t; const void* v_t;          // bf16 [B][H][128]
  uint8_t* k_cache; uint8_t* v_cache;                       // [B][H][cap][128] bytes
  const float* k_scale; const float* v_scale;               // [H]
  const int32_t* cache_len; const uint8_t* keep;
  void* out;                                                // bf16 [B][H][128]
  float* partial; int32_t* ticket; DeviceStatus* status;
  int32_t B, H, cap, per_bh, slots, n_stages;
  int32_t overlap;        // launched with programmatic stream serialisation: may start while its predecessor drains
  float scale_log2;
};

__device__ __forceinline__ int f8_chunks(int n, const F8Args& a) {
  return max(1, min(a.per_bh, n / kDecodeMinChunk));
}

struct F8Item { int b, h, c, nch, n_b, r0, rows, nst; };

__device__ __forceinline__ void f8_ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void f8_ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// two E4M3 bytes (the low 16 bits of v) -> an fp16 pair
__device__ __forceinline__ uint32_t f8_pair_to_f16x2(uint32_t v) {
  uint32_t r;
  asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %1; cvt.rn.f16x2.e4m3x2 %0, lo; }" : "=r"(r) : "r"(v));
  return r;
}
__device__ __forceinline__ uint32_t f8_hi_pair_to_f16x2(uint32_t v) {
  uint32_t r;
  asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %1; cvt.rn.f16x2.e4m3x2 %0, hi; }" : "=r"(r) : "r"(v));
  return r;
}
// bytes 0 and 2 of v (prmt 0x..20) or bytes 1 and 3 (0x..31) into the low half
__device__ __forceinline__ uint32_t f8_even_bytes(uint32_t v) { return __byte_perm(v, 0u, 0x4420); }
__device__ __forceinline__ uint32_t f8_odd_bytes(uint32_t v) { return __byte_perm(v, 0u, 0x4431); }
// two floats -> an fp16 pair (low half first)
__device__ __forceinline__ uint32_t f8_pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// two floats -> two E4M3 bytes (low byte first), round to nearest even, clamped to +-448
__device__ __forceinline__ uint32_t f8_encode_pair(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// D += A (16 x 16 fp16, only row 0 of the fragment can be non-zero here) * B (16 x 8 fp16)
__device__ __forceinline__ void f8_mma(float* c, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void f8_tma_2d(uint32_t dst, const void* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t f8_pack_bf16x2(float lo, float hi) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}

struct F8Maps { alignas(64) unsigned char k[128]; alignas(64) unsigned char v[128]; };

__global__ void __launch_bounds__(kF8Warps * 32, kF8Ctas)
attn_decode_fp8_kernel(const __grid_constant__ F8Maps maps, const F8Args a) {
  constexpr int D = 128, RB = 256, RS = kF8Rows;      // RB: bytes of a bf16 row (q, k_t, v_t, out)
  extern __shared__ char smem_raw[];
  char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NS = a.n_stages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  char* my_tiles = smem + (size_t)warp * NS * kF8Stage;
  uint64_t* all_bars = reinterpret_cast<uint64_t*>(smem + (size_t)kF8Warps * NS * kF8Stage);
  uint64_t* bars = all_bars + warp * NS;
  int* prefix = reinterpret_cast<int*>(all_bars + kF8Warps * NS);
  __shared__ int sh_abort;
  volatile int* abort_flag = &sh_abort;

  // Let the next kernel of the stream start as soon as SMs free up (it only matters when that kernel was launched
  // with programmatic stream serialisation; a no-op otherwise).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) sh_abort = 0;
  if (lane == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_mbar_init();
  }
  for (int b = tid; b < a.B; b += kF8Warps * 32) {
    int n = min(max(a.cache_len[b], 0), a.cap);
    prefix[b + 1] = f8_chunks(n, a) * a.H;
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    prefix[0] = 0;
    for (int b = 0; b < a.B; ++b) { run += prefix[b + 1]; prefix[b + 1] = run; }
  }
  __syncthreads();
  const int total = prefix[a.B];
  const int GW = gridDim.x * kF8Warps;
  const int gw = (total >= GW) ? blockIdx.x * kF8Warps + warp : warp * gridDim.x + blockIdx.x;

  auto load_item = [&](int item, F8Item& I) {
    int lo = 0, hi = a.B - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (prefix[mid] <= item) lo = mid; else hi = mid - 1;
    }
    I.b = lo;
    I.n_b = min(max(a.cache_len[lo], 0), a.cap);
    I.nch = f8_chunks(I.n_b, a);
    const int r = item - prefix[lo];
    I.h = r / I.nch;
    I.c = r - I.h * I.nch;
    const int cs = ((I.n_b + I.nch - 1) / I.nch + RS - 1) / RS * RS;
    I.r0 = I.c * cs;
    I.rows = max(0, min(I.n_b, I.r0 + cs) - I.r0);
    I.nst = max(1, (I.rows + RS - 1) / RS);
  };
  // lane 0: whole 32-row boxes are fetched even for a ragged last tile (the surplus rows are masked);
  // rows past the end of the tensor read as zero
  auto issue = [&](const F8Item& I, int st, int slot) {
    const uint32_t full = smem_u32(&bars[slot]);
    if (I.rows - st * RS <= 0) { mbar_arrive(full); return; }
    const int row0 = (I.b * a.H + I.h) * a.cap + I.r0 + st * RS;
    mbar_expect_tx(full, kF8Stage);
    const uint32_t dst = smem_u32(my_tiles + (size_t)slot * kF8Stage);
    f8_tma_2d(dst, maps.k, 0, row0, full);
    f8_tma_2d(dst + kF8Box, maps.v, 0, row0, full);
  };

  int p_item = gw, p_st = 0, issued = 0, consumed = 0;
  F8Item PI;
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

  // ---- registers fetched one item ahead.  Lane t (< 4) owns, of each 16-dim chunk c, dims 16c + 4t .. 16c + 4t + 3:
  //      as the A operand of q K^T (see the file header) and as the output columns of P V.
  const int t4 = lane & 3;
  const bool row0_lane = lane < 4;
  uint2 nq[8], nk[8];                                 // raw bf16 quads of q and k_t, per chunk
  uint2 nks, nvs;                                     // this lane's 4 dims (4 lane .. 4 lane + 3) of k_t, v_t for the append
  auto prefetch = [&](const F8Item& I) {
    const size_t off = ((size_t)I.b * a.H + I.h) * RB;
    const char* qb = (const char*)a.q + off;
    const char* kb = (const char*)a.k_t + off;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      nq[c] = row0_lane ? __ldg(reinterpret_cast<const uint2*>(qb + (16 * c + 4 * t4) * 2)) : make_uint2(0u, 0u);
      nk[c] = row0_lane ? __ldg(reinterpret_cast<const uint2*>(kb + (16 * c + 4 * t4) * 2)) : make_uint2(0u, 0u);
    }
    nks = __ldg(reinterpret_cast<const uint2*>(kb + lane * 8));
    nvs = __ldg(reinterpret_cast<const uint2*>((const char*)a.v_t + off + lane * 8));
  };
  F8Item I, NI;
  if (gw < total) { load_item(gw, NI); prefetch(NI); }

  // ldmatrix lane addressing: lane -> (matrix m = lane / 8, row r = lane % 8)
  const int lm = lane >> 3, lr = lane & 7;
  const int k_row = (lm >> 1) * 8 + lr, k_csel = lm & 1;      // q K^T: matrices 0,1 keys 0-7 (chunks c, c+1); 2,3 keys 8-15
  const int v_row = (lm & 1) * 8 + lr, v_csel = lm >> 1;      // P V:   matrices 0,1 keys 0-7 / 8-15 of chunk c; 2,3 of chunk c+1

  for (int item = gw; item < total; item += GW) {
    I = NI;
    const size_t bh = (size_t)I.b * a.H + I.h;
    const float ks_log2 = __ldg(a.k_scale + I.h) * a.scale_log2;      // scores: (q . bytes) * k_scale * scale, base 2
    const float v_scale = __ldg(a.v_scale + I.h);
    uint32_t qa[16];
    float s_e = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      qa[2 * c] = f8_pack_f16x2(bf16lo(nq[c].x), bf16hi(nq[c].x));
      qa[2 * c + 1] = f8_pack_f16x2(bf16lo(nq[c].y), bf16hi(nq[c].y));
      s_e = fmaf(bf16lo(nq[c].x), bf16lo(nk[c].x), s_e);
      s_e = fmaf(bf16hi(nq[c].x), bf16hi(nk[c].x), s_e);
      s_e = fmaf(bf16lo(nq[c].y), bf16lo(nk[c].y), s_e);
      s_e = fmaf(bf16hi(nq[c].y), bf16hi(nk[c].y), s_e);
    }
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 1);
    s_e += __shfl_xor_sync(0xffffffffu, s_e, 2);
    s_e = __shfl_sync(0xffffffffu, s_e, 0) * a.scale_log2;
    if (I.c == 0 && a.keep != nullptr && a.keep[I.b] != 0) {
      if (I.n_b < a.cap) {
        // the kept token's row as bytes: x / scale in fp32, nearest code, clamped; 4 dims per lane
        const float ksc = __ldg(a.k_scale + I.h);
        const size_t dst = (bh * a.cap + I.n_b) * 128 + lane * 4;
        const uint32_t kb = f8_encode_pair(__fdiv_rn(bf16lo(nks.x), ksc), __fdiv_rn(bf16hi(nks.x), ksc)) |
                            (f8_encode_pair(__fdiv_rn(bf16lo(nks.y), ksc), __fdiv_rn(bf16hi(nks.y), ksc)) << 16);
        const uint32_t vb = f8_encode_pair(__fdiv_rn(bf16lo(nvs.x), v_scale), __fdiv_rn(bf16hi(nvs.x), v_scale)) |
                            (f8_encode_pair(__fdiv_rn(bf16lo(nvs.y), v_scale), __fdiv_rn(bf16hi(nvs.y), v_scale)) << 16);
        if (DL_IN_BOUNDS(a.status, KID_DECODE_FP8, dst + 3, (size_t)a.B * a.H * a.cap * 128)) {
          *reinterpret_cast<uint32_t*>(a.k_cache + dst) = kb;
          *reinterpret_cast<uint32_t*>(a.v_cache + dst) = vb;
        }
      } else if (lane == 0 && I.h == 0) {
        report_status(a.status, DL_ERR_CAPACITY, I.b);
      }
    }
    if (item + GW < total) { load_item(item + GW, NI); prefetch(NI); }

    float m_run = -INFINITY, l_run = 0.f;          // l_run: this lane's share of the sum
    float accE[8][4], accO[8][4];                  // chunk c: even / odd dims; [0], [1] are row 0 (lanes 0-3)
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      accE[c][0] = accE[c][1] = accE[c][2] = accE[c][3] = 0.f;
      accO[c][0] = accO[c][1] = accO[c][2] = accO[c][3] = 0.f;
    }

    for (int st = 0; st < I.nst; ++st, ++consumed) {
      const int slot = consumed % NS;
      mbar_wait(smem_u32(&bars[slot]), (consumed / NS) & 1, abort_flag);
      const int nr = min(RS, I.rows - st * RS);
      if (nr > 0) {
        const uint32_t tile = smem_u32(my_tiles + (size_t)slot * kF8Stage);
        if (nr < RS) {
          // ragged last tile: rows >= nr hold unrelated bytes (possibly NaN codes); zero them in V so that 0 * x stays 0
          char* vz = my_tiles + (size_t)slot * kF8Stage + kF8Box;
          for (int u = lane; u < RS * 8; u += 32) {
            const int r = u >> 3;
            if (r >= nr) *reinterpret_cast<uint4*>(vz + r * 128 + (u & 7) * 16) = make_uint4(0, 0, 0, 0);
          }
          __syncwarp();
        }
        // ---- S = q . K^T for 32 rows: four blocks of 8 keys
        float s[4][4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
#pragma unroll
          for (int cp = 0; cp < 4; ++cp) {
            const int row = kb * 16 + k_row, chunk = 2 * cp + k_csel;
            const uint32_t addr = tile + row * 128 + (((chunk) ^ (row & 7)) << 4);
            uint32_t r0, r1, r2, r3;
            f8_ldsm_x4(addr, r0, r1, r2, r3);
            const int c = 2 * cp;
            f8_mma(s[2 * kb], qa[2 * c], qa[2 * c + 1], f8_pair_to_f16x2(r0), f8_hi_pair_to_f16x2(r0));
            f8_mma(s[2 * kb], qa[2 * c + 2], qa[2 * c + 3], f8_pair_to_f16x2(r1), f8_hi_pair_to_f16x2(r1));
            f8_mma(s[2 * kb + 1], qa[2 * c], qa[2 * c + 1], f8_pair_to_f16x2(r2), f8_hi_pair_to_f16x2(r2));
            f8_mma(s[2 * kb + 1], qa[2 * c + 2], qa[2 * c + 3], f8_pair_to_f16x2(r3), f8_hi_pair_to_f16x2(r3));
          }
        }
        // ---- online softmax; lanes 0-3 hold keys 8 nb + 2t, 8 nb + 2t + 1 of block nb
        float sv[8];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
          sv[2 * nb] = (row0_lane && 8 * nb + 2 * t4 < nr) ? s[nb][0] * ks_log2 : -INFINITY;
          sv[2 * nb + 1] = (row0_lane && 8 * nb + 2 * t4 + 1 < nr) ? s[nb][1] * ks_log2 : -INFINITY;
        }
        float mx = fmaxf(fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3])), fmaxf(fmaxf(sv[4], sv[5]), fmaxf(sv[6], sv[7])));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        mx = __shfl_sync(0xffffffffu, mx, 0);
        if (mx > m_run) {                                            // warp-uniform
          const float corr = exp2f(m_run - mx);
          l_run *= corr;
#pragma unroll
          for (int c = 0; c < 8; ++c) { accE[c][0] *= corr; accE[c][1] *= corr; accO[c][0] *= corr; accO[c][1] *= corr; }
          m_run = mx;
        }
        float p[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { p[i] = exp2f(sv[i] - m_run); l_run += p[i]; }
        // ---- O += P . V : per 16 keys, per 16-dim chunk, one MMA over the even and one over the odd dims
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint32_t pa0 = f8_pack_f16x2(p[4 * kb], p[4 * kb + 1]), pa2 = f8_pack_f16x2(p[4 * kb + 2], p[4 * kb + 3]);
#pragma unroll
          for (int cp = 0; cp < 4; ++cp) {
            const int row = kb * 16 + v_row, chunk = 2 * cp + v_csel;
            const uint32_t addr = tile + kF8Box + row * 128 + (((chunk) ^ (row & 7)) << 4);
            uint32_t r0, r1, r2, r3;
            f8_ldsm_x4_t(addr, r0, r1, r2, r3);
            const int c = 2 * cp;
            f8_mma(accE[c], pa0, pa2, f8_pair_to_f16x2(f8_even_bytes(r0)), f8_pair_to_f16x2(f8_even_bytes(r1)));
            f8_mma(accO[c], pa0, pa2, f8_pair_to_f16x2(f8_odd_bytes(r0)), f8_pair_to_f16x2(f8_odd_bytes(r1)));
            f8_mma(accE[c + 1], pa0, pa2, f8_pair_to_f16x2(f8_even_bytes(r2)), f8_pair_to_f16x2(f8_even_bytes(r3)));
            f8_mma(accO[c + 1], pa0, pa2, f8_pair_to_f16x2(f8_odd_bytes(r2)), f8_pair_to_f16x2(f8_odd_bytes(r3)));
          }
        }
        if (nr < RS) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      __syncwarp();
      if (p_valid && !*abort_flag) {
        if (lane == 0) issue(PI, p_st, slot);
        advance_producer();
      }
    }

    // ---- finish the item: lanes 0-3 own the output; of chunk c lane t has dims 16c + 4t .. 16c + 4t + 3 as
    //      (accE[c][0], accO[c][0], accE[c][1], accO[c][1]); the cached part carries v_scale
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    l_run = __shfl_sync(0xffffffffu, l_run, 0);
    char* outb = (char*)a.out + bh * RB;
    const char* vtb = (const char*)a.v_t + bh * RB;
    if (I.nch == 1) {
      const float M2 = fmaxf(m_run, s_e);
      const float wn = (m_run == -INFINITY) ? 0.f : exp2f(m_run - M2);
      const float we = exp2f(s_e - M2);
      const float inv = 1.f / (l_run * wn + we);
      const float wc = wn * v_scale;
      if (row0_lane && DL_IN_BOUNDS(a.status, KID_DECODE_FP8, bh * RB + RB - 1, (size_t)a.B * a.H * RB)) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint2 vw = __ldg(reinterpret_cast<const uint2*>(vtb + (16 * c + 4 * t4) * 2));
          uint2 o;
          o.x = f8_pack_bf16x2((accE[c][0] * wc + we * bf16lo(vw.x)) * inv, (accO[c][0] * wc + we * bf16hi(vw.x)) * inv);
          o.y = f8_pack_bf16x2((accE[c][1] * wc + we * bf16lo(vw.y)) * inv, (accO[c][1] * wc + we * bf16hi(vw.y)) * inv);
          *reinterpret_cast<uint2*>(outb + (16 * c + 4 * t4) * 2) = o;
        }
      }
      continue;
    }
    // a sequence split over several items: partial sums (with v_scale applied) in dim order, merged by the last to arrive
    float* part = a.partial + (bh * a.slots + I.c) * (size_t)(D + 2);
    if (row0_lane) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {                 // a slot is 130 floats: 8-byte, not 16-byte, aligned
        *reinterpret_cast<float2*>(part + 16 * c + 4 * t4) = make_float2(accE[c][0] * v_scale, accO[c][0] * v_scale);
        *reinterpret_cast<float2*>(part + 16 * c + 4 * t4 + 2) = make_float2(accE[c][1] * v_scale, accO[c][1] * v_scale);
      }
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
      for (int c = 0; c < 8; ++c) {
        const uint2 vw = row0_lane ? __ldg(reinterpret_cast<const uint2*>(vtb + (16 * c + 4 * t4) * 2)) : make_uint2(0u, 0u);
        num[4 * c] = we * bf16lo(vw.x);
        num[4 * c + 1] = we * bf16hi(vw.x);
        num[4 * c + 2] = we * bf16lo(vw.y);
        num[4 * c + 3] = we * bf16hi(vw.y);
      }
      for (int cc = 0; cc < I.nch; ++cc) {
        const float* pc = p0 + (size_t)cc * (D + 2);
        const float mc = __ldcg(pc + D);
        const float wt = (mc == -INFINITY) ? 0.f : exp2f(mc - Mg);
        den = fmaf(__ldcg(pc + D + 1), wt, den);
        if (row0_lane) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const float2 va = __ldcg(reinterpret_cast<const float2*>(pc + 16 * c + 4 * t4));
            const float2 vb = __ldcg(reinterpret_cast<const float2*>(pc + 16 * c + 4 * t4 + 2));
            num[4 * c] = fmaf(va.x, wt, num[4 * c]);
            num[4 * c + 1] = fmaf(va.y, wt, num[4 * c + 1]);
            num[4 * c + 2] = fmaf(vb.x, wt, num[4 * c + 2]);
            num[4 * c + 3] = fmaf(vb.y, wt, num[4 * c + 3]);
          }
        }
      }
      const float inv = 1.f / den;
      if (row0_lane) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint2 o;
          o.x = f8_pack_bf16x2(num[4 * c] * inv, num[4 * c + 1] * inv);
          o.y = f8_pack_bf16x2(num[4 * c + 2] * inv, num[4 * c + 3] * inv);
          *reinterpret_cast<uint2*>(outb + (16 * c + 4 * t4) * 2) = o;
        }
      }
      if (lane == 0) a.ticket[bh] = 0;
    }
  }

  // A kernel that was allowed to start early must not finish before its predecessor has: whatever follows in the
  // stream relies on all earlier layers being done.
  if (a.overlap) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (*abort_flag) {
    if (lane == 0) {
      report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
      for (int j = max(0, issued - NS); j < issued; ++j)
        for (int i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&bars[j % NS]), (j / NS) & 1); ++i) __nanosleep(40);
    }
  }
}

// Rows [0, cache_len[b]) of a bf16 cache [B][H][cap][128] as E4M3 bytes under per-head scales: x / scale in fp32,
// nearest code (ties to even), clamped to +-448.  One thread per 8 elements.
__global__ void quantize_kv_fp8_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ cache_len,
                                       const float* __restrict__ scale, int32_t H, int32_t cap, long long n8,
                                       uint2* __restrict__ dst, DeviceStatus* st) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n8) return;
  const long long row = i >> 4;                     // 16 groups of 8 per 128-dim row
  const int r = (int)(row % cap);
  const long long bh = row / cap;
  const int h = (int)(bh % H), b = (int)(bh / H);
  if (r >= min(max(cache_len[b], 0), cap)) return;
  const float sc = __ldg(scale + h);
  const uint4 v = __ldg(src + i);
  uint2 o;
  o.x = f8_encode_pair(__fdiv_rn(bf16lo(v.x), sc), __fdiv_rn(bf16hi(v.x), sc)) |
        (f8_encode_pair(__fdiv_rn(bf16lo(v.y), sc), __fdiv_rn(bf16hi(v.y), sc)) << 16);
  o.y = f8_encode_pair(__fdiv_rn(bf16lo(v.z), sc), __fdiv_rn(bf16hi(v.z), sc)) |
        (f8_encode_pair(__fdiv_rn(bf16lo(v.w), sc), __fdiv_rn(bf16hi(v.w), sc)) << 16);
  if (DL_IN_BOUNDS(st, KID_QUANTIZE, i, n8)) dst[i] = o;
}

cudaError_t launch_quantize_kv_fp8(const dl_ctx* ctx, const void* src, const int32_t* cache_len, const float* scale,
                                   int32_t B, int32_t cap, void* dst, cudaStream_t s) {
  const long long n8 = (long long)B * ctx->desc.n_heads * cap * 16;
  if (n8 == 0) return cudaSuccess;
  const long long blocks = (n8 + 255) / 256;
  if (blocks >= (1LL << 31)) return cudaErrorInvalidValue;
  quantize_kv_fp8_kernel<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const uint4*>(src), cache_len, scale,
                                                           ctx->desc.n_heads, cap, n8, static_cast<uint2*>(dst),
                                                           ctx->ws.base ? ctx->ws.status : nullptr);
  return cudaGetLastError();
}

static int f8_max_chunks(const F8Args& a) { return max(1, min(a.per_bh, a.cap / kDecodeMinChunk)); }

cudaError_t launch_attn_decode_fp8(const dl_ctx* ctx, const void* q, const void* k_t, const void* v_t, void* k_cache,
                                   void* v_cache, const float* k_scale, const float* v_scale, const int32_t* cache_len,
                                   const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                                   cudaStream_t s, bool in_stack, bool overlap_prev, int scratch_set) {
  if (B == 0) return cudaSuccess;
  const dl_model_desc& d = ctx->desc;
  if (d.dtype != DL_BF16 || d.head_dim != 128 || ctx->tmap_encode == nullptr) return cudaErrorInvalidValue;
  F8Args a;
  a.q = q; a.k_t = k_t; a.v_t = v_t;
  a.k_cache = static_cast<uint8_t*>(k_cache); a.v_cache = static_cast<uint8_t*>(v_cache);
  a.k_scale = k_scale; a.v_scale = v_scale; a.cache_len = cache_len; a.keep = keep; a.out = out;
  // the scratch of split sequences: one of three sets, so that launches in flight together differ (see
  // launch_attn_decode for why three are enough)
  const size_t set = (size_t)(scratch_set % kDecodeScratchSets);
  a.ticket = ctx->ws.dec_ticket + set * (size_t)ctx->ws.max_batch * d.n_heads;
  a.partial = ctx->ws.dec_partial + set * (size_t)ctx->ws.max_batch * d.n_heads * ctx->ws.dec_slots * (d.head_dim + 2);
  a.status = ctx->ws.status;
  a.B = B; a.H = d.n_heads; a.cap = cap; a.slots = ctx->ws.dec_slots;
  const long long warps = (long long)ctx->sm_count * kF8Warps * kF8Ctas;
  a.per_bh = (int)max(1LL, warps / ((long long)B * d.n_heads));
  a.scale_log2 = scale * 1.4426950408889634f;
  // the bytes of a cache row seen as 64 two-byte elements: [B*H*cap rows][128 bytes], box 32 rows, 128-byte swizzle
  F8Maps maps;
  const long long rows = (long long)B * d.n_heads * cap;
  if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
  const uint64_t dims[2] = {64ull, (uint64_t)rows};
  const uint64_t strides[1] = {128ull};
  const uint32_t box[2] = {64u, (uint32_t)kF8Rows};
  if (!encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps.k), k_cache, 2, dims, strides, box) ||
      !encode_bf16_map(ctx->tmap_encode, reinterpret_cast<CUtensorMap*>(maps.v), v_cache, 2, dims, strides, box))
    return cudaErrorInvalidValue;
  const size_t fixed = (size_t)(B + 1) * sizeof(int) + 1024 /*alignment*/ + 256;
  const int per_cta = (ctx->smem_optin + 1024) / kF8Ctas - 1024;
  int ns = (int)((per_cta - 256 - (int)fixed) / (kF8Warps * (kF8Stage + 8)));
  ns = min(ns, 6);
  if (ns < 2) return cudaErrorInvalidConfiguration;
  a.n_stages = ns;
  const size_t smem = (size_t)kF8Warps * ns * (kF8Stage + 8) + fixed;
  static int attr_set[64];
  int& attr_set_for = attr_set[ctx->device & 63];
  if (attr_set_for != (int)smem) {
    cudaError_t e = cudaFuncSetAttribute(attn_decode_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set_for = (int)smem;
  }
  const long long max_items = (long long)B * d.n_heads * f8_max_chunks(a);
  // Inside a layer stack a launch takes ONE of the two CTA slots of an SM and may start while its predecessor
  // drains, so that two layers stream side by side (as the bf16 kernel does); that counts on exactly two CTAs of
  // this kernel fitting an SM.
  static int occ_for[64], occ_val[64];
  if (occ_for[ctx->device & 63] != (int)smem) {
    int nb = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, attn_decode_fp8_kernel, kF8Warps * 32, smem);
    if (e != cudaSuccess) return e;
    occ_val[ctx->device & 63] = nb;
    occ_for[ctx->device & 63] = (int)smem;
  }
  const bool one_slot = in_stack && max_items >= ctx->sm_count && occ_val[ctx->device & 63] == kF8Ctas;
  a.overlap = (overlap_prev && (one_slot || f8_max_chunks(a) == 1)) ? 1 : 0;
  const int grid = (int)max(1LL, min((long long)ctx->sm_count * (one_slot ? 1 : kF8Ctas), max_items));
  if (!a.overlap) {
    attn_decode_fp8_kernel<<<grid, kF8Warps * 32, smem, s>>>(maps, a);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kF8Warps * 32); cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attn_decode_fp8_kernel, maps, a);
}

}  // namespace dl
