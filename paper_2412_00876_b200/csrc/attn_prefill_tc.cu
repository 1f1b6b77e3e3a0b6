// Prefill attention over the reduced set on the tensor cores (Eq. 1 applied to S^{P*}):
// row i of a sequence's compact context attends rows 0..i of the same context.
// bf16, head_dim 128.  One persistent CTA per SM walks work items (sequence, head, PAIR of 128-row query tiles),
// longest pairs first.  The two query tiles of a pair go to the CTA's two lanes, A (the later rows) and B (the 128
// rows before them; the lanes swap from one item to the next so that they do the same work).  A lane is a pipeline
// of its own: its Q, K and V slots in shared memory, its score / output accumulators in tensor memory, its
// MMA-issuing thread and its four softmax warps.  Pairs are aligned to the END of a sequence (rows
// [n-256(p+1), n-256p)), so the ragged pair is the one at the top of the causal triangle, where it needs the fewest
// keys; lane B of a pair that has 128 rows or fewer does not exist and the lane moves on to the next item.
// Every lane fetches its OWN K and V tiles: a lane whose tile has fewer key tiles than its partner's finishes its
// item and starts the next one at once.  (With one K/V ring shared by the lanes, each tile fetched once per pair,
// the shorter lane waited at the ring for the longer one to release a slot; K and V now cross from L2 into shared
// memory once per query tile, which measured no slower at any context length.)
// Shared memory, 7 tiles of 32 KB: per lane a Q slot, a K slot and a V slot; the seventh tile is the lanes' output
// staging (16 KB each).
// There is NO producer role: a slot is refilled by the first thread of one of the lane's softmax warps at the moment
// that thread learns the slot is free, which it learns anyway.  "S_u is ready" is a commit behind P_{u-1} V_{u-1} and
// Q K_u^T, so when that wait ends the K slot (K_u has been read) and the V slot (V_{u-1} has been read) are both free:
// K_{u+1} and V_u are requested there, then the warps run the softmax of S_u, which is what hides the copies; behind
// the item's last Q K^T the Q slot is free too and the next item's Q and K_0 are requested; "O is complete" (behind the
// item's last P V) frees the V slot for the next item's V_0.  A polling producer thread took 2-5 k cycles from a
// slot's release to the request (its code is cold at every use and it competes with the softmax warps for issue
// slots), which a one-deep slot cannot hide; here that delay is a few instructions.
//   warps 9,10 : the MMA-issuing thread of lane A / B:
//                S = Q K^T (128 x N, K-major operands from shared memory), O += P V (P read from tensor memory, V
//                as an MN-major shared-memory operand).  Block u = P_u V_u then Q K_{u+1}^T (which overwrites P: in
//                order behind the P V), one commit set per block.  Full tiles use N = 128 keys; a lane's last tile
//                uses N = keys left rounded up to 16, in both products.
//   warps 0-3 / 4-7 : softmax of lane A / B, one query row per thread, straight out of tensor memory in 32-column
//                chunks (these warps take the registers the other warps give back); chunks that no row of the
//                warp may see (above the causal diagonal) are skipped.  The running maximum is only raised when a
//                chunk's maximum exceeds it by more than 2^8 (then O is rescaled in tensor memory), so most tiles
//                never touch O.  P (bf16) overwrites the first half of S.  First threads of three of the warps: the
//                lane's TMA requests.  The same warps normalise O and store it: 32 x 32 blocks staged in the lane's
//                staging area, two column blocks at a time, sent with TMA stores (predicated stores for a tile
//                clipped at the top of a sequence, whose surplus rows belong to the next tile).
//   warp 11    : tensor-memory allocation (all 512 columns: O_A | S_A | O_B | S_B), then the top rows of sequences
//                whose length leaves a top tile of at most 16 rows (attn_prefill_top.cuh), which the lanes skip
//   warp 8     : idle
// Barrier phases follow running counters per lane (its key tiles g, its items i): tile g completes phase g & 1 of
// k_full / v_full / s_full / p_full / pv_done; item i phase i & 1 of q_full / o_free.  No waiter can be two phases
// behind: K tile g + 1 is only requested once the Q K^T of tile g has completed, and so on round the cycle.
// Rows past a sequence's length are fetched with the tile (they are masked); where the 16-row rounding of the last
// tile reaches past the sequence's end, those V rows are zeroed in shared memory first, since 0 * x must stay 0 for
// any bit pattern.  Every wait is bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

#include "attn_prefill.cuh"
#include "attn_prefill_softmax.cuh"
#include "attn_prefill_top.cuh"

namespace dl {

constexpr int kAtLaneTiles = 3;                         // Q, K, V slot of a lane
constexpr int kAtTurnTiles = 4;                         // items of at least this many key tiles take turns at the softmax
constexpr int kAtOffStage = 2 * kAtLaneTiles * kAtTile; // 16 KB of staging per lane
static_assert(kAtOffStage + kAtTile == kAtOffBar, "seven tiles, then the barriers");

__global__ void __launch_bounds__(kAtThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ AtMaps maps, const AtArgs a) {
  extern __shared__ __align__(1024) char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (smem_u32(smem) & 1023u) {                        // the swizzled tiles need 1024-byte alignment
    if (tid == 0) report_status(a.status, DL_ERR_ALIGNMENT, -1);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAtOffBar);
  auto slot = [&](int x, int which) { return smem + (x * kAtLaneTiles + which) * kAtTile; };   // 0 Q, 1 K, 2 V
  auto bar = [&](int x, int i) { return smem_u32(bars + 16 * x + i); };
  enum { Q_FULL = 0, K_FULL, V_FULL, S_FULL, P_FULL, PV_DONE, O_FREE };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 33);
  volatile int* in_softmax = reinterpret_cast<volatile int*>(bars + 36);     // [lane x][warp quad]: see the softmax role

  if (tid == 0) {
    *abort_flag = 0;
    for (int i = 0; i < 8; ++i) in_softmax[i] = 0;
    for (int x = 0; x < 2; ++x) {
      for (int i = Q_FULL; i <= O_FREE; ++i) mbar_init(bar(x, i), (i == P_FULL || i == O_FREE) ? 4 : 1);
    }
    fence_mbar_init();
  }
  if (warp == 11) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 9 || warp == 10) {
    // ---------------------------------------------------------------- MMA issuer of one lane
    reg_dec<kAtRegsSmall>();
    if (lane == 0) {
      const int x = warp - 9;
      const uint32_t t_o = tmem + x * kAtLaneCols + kAtColO, t_s = tmem + x * kAtLaneCols + kAtColS;
      const uint32_t idesc_pv = idesc_bf16(kAtBM, 128, 0, 1);          // B (= V) is MN-major
      const uint64_t q_desc = smem_desc_sw128(smem_u32(slot(x, 0)));
      const uint64_t k_desc = smem_desc_sw128(smem_u32(slot(x, 1)));
      const uint64_t v_desc0 = smem_desc_sw128_mn(smem_u32(slot(x, 2)), kAtBN * 128);
      AtWalker W(a);
      AtItem I;
      int n_item = 0, g0 = 0;                         // this lane's items / key tiles so far
      while (W.next(I, kAtTopRows)) {
        const AtLane L = at_lane(I, x);
        if (!L.exists) continue;
        const int n_sub = L.n_tiles;
        // Block u of the item: O += P_u V_u, then S = Q K_{u+1}^T (which overwrites P: in order behind the P V).
        // Block -1 is the first Q K^T alone (it may run while the previous item's output is still being read
        // out of O), the last block the last P V alone.  One rolled copy of the code for all of them.
        for (int u = -1; u < n_sub; ++u) {
          const int g = g0 + u;
          const bool has_pv = u >= 0, has_qk = u + 1 < n_sub;
          if (has_pv) mbar_wait_spin(bar(x, V_FULL), (uint32_t)g & 1u, abort_flag);
          else mbar_wait_spin(bar(x, Q_FULL), (uint32_t)n_item & 1u, abort_flag);
          if (has_qk) mbar_wait_spin(bar(x, K_FULL), (uint32_t)(g + 1) & 1u, abort_flag);
          if (u == 0) mbar_wait_spin(bar(x, O_FREE), ((uint32_t)n_item & 1u) ^ 1u, abort_flag);   // previous item's O has been read
          if (has_pv) mbar_wait_spin(bar(x, P_FULL), (uint32_t)g & 1u, abort_flag);
          tc_fence_after();
          if (has_pv) {
            uint64_t vd = v_desc0;
            const int ksteps = at_cols(L, u) >> 4;
#pragma unroll 1
            for (int ks = 0; ks < ksteps; ++ks, vd += 2048 >> 4)
              mma_ts(t_o, t_s + ks * 8, vd, idesc_pv, (u | ks) != 0);
          }
          if (has_qk) {
            // 16 dims further per step, and from the fourth step on in the tile's second 64-dim half
            uint64_t qd = q_desc, kd = k_desc;
            const uint32_t idesc_qk = idesc_bf16(kAtBM, (uint32_t)at_cols(L, u + 1));
#pragma unroll 1
            for (int ks = 0; ks < 8; ++ks) {
              mma_ss(t_s, qd, kd, idesc_qk, ks != 0);
              const uint64_t step = (ks == 3) ? (uint64_t)((kAtBM * 128 - 96) >> 4) : 2ull;
              qd += step;
              kd += step;
            }
            mma_commit(bar(x, S_FULL));          // the softmax warps wait on it; it also frees the K and V slots
          }
          if (has_pv) mma_commit(bar(x, PV_DONE));
        }
        g0 += n_sub;
        ++n_item;
      }
    }
  } else if (warp < 8) {
    // ---------------------------------------------------------------- softmax / epilogue warps of one lane
    reg_inc<kAtRegsSoftmax>();
    const int x = warp >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                                  // row within the query tile
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const uint32_t s_addr = tmem + lane_off + x * kAtLaneCols + kAtColS;
    const uint32_t o_addr = tmem + lane_off + x * kAtLaneCols + kAtColO;
    const CUtensorMap* mo = reinterpret_cast<const CUtensorMap*>(maps.o);
    char* so = smem + kAtOffStage + x * (kAtTile / 2) + quad * 4096;   // this warp's 4 KB: two 32 x 32 blocks
    // ---- this lane's TMA requests
    // (a request costs its thread about 300 cycles, so the three kinds go to three warps' first threads)
    const bool issue_k = quad == 0 && lane == 0, issue_v = quad == 1 && lane == 0, issue_q = quad == 2 && lane == 0;
    int issued[3] = {0, 0, 0};                                         // Q / K / V copies requested so far by this thread
    auto load_q = [&](const AtItem& It, const AtLane& Ln) {
      // the rows the lane owns, in 16s (a tile clipped at the top of the sequence owns fewer than 128)
      const int bx = at_box(min(kAtBM, (Ln.q_hi - Ln.q0 + 15) & ~15));
      const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(maps.q[bx]);
      char* dst = slot(x, 0);
      mbar_expect_tx(bar(x, Q_FULL), kAtTile >> bx);
      tma_load_2d(smem_u32(dst), mq, 0, It.row_base + Ln.q0, bar(x, Q_FULL));
      tma_load_2d(smem_u32(dst + kAtBM * 128), mq, 64, It.row_base + Ln.q0, bar(x, Q_FULL));
      ++issued[0];
    };
    auto load_kv = [&](const AtItem& It, const AtLane& Ln, int j, int is_v) {
      const int bx = at_box(at_cols(Ln, j));                           // keys of the tile that this lane covers
      const CUtensorMap* m = reinterpret_cast<const CUtensorMap*>(is_v ? maps.v[bx] : maps.k[bx]);
      char* dst = slot(x, 1 + is_v);
      const uint32_t fb = bar(x, is_v ? V_FULL : K_FULL);
      const int r = It.row_base + j * kAtBN;
      mbar_expect_tx(fb, kAtTile >> bx);
      tma_load_2d(smem_u32(dst), m, 0, r, fb);
      tma_load_2d(smem_u32(dst + kAtBN * 128), m, 64, r, fb);
      ++issued[1 + is_v];
    };
    AtWalker W(a);
    AtItem I, In, In2;                                                 // this item, the next, the one after
    AtLane L, Ln, Ln2;
    auto next_own = [&](AtItem& It, AtLane& Lt) {                      // the next item in which this lane has a tile
      while (W.next(It, kAtTopRows)) {
        Lt = at_lane(It, x);
        if (Lt.exists) return true;
      }
      return false;
    };
    if (lane == 0 && quad < 3) {
      const unsigned char (*mp)[128] = issue_q ? maps.q : issue_k ? maps.k : maps.v;
      for (int i = 0; i < 4; ++i) tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(mp[i]));
    }
    // The walk runs two items ahead: the step to item i + 2 is taken while item i waits for its last P V (idle time;
    // at the top of the loop it would sit in front of the first softmax, 1 k cycles of cold code per item).
    bool have = next_own(I, L);
    bool have_next = have && next_own(In, Ln);
    if (have) {
      if (issue_q) load_q(I, L);
      if (issue_k) load_kv(I, L, 0, 0);
      if (issue_v) load_kv(I, L, 0, 1);
    }
    int g0 = 0;
    while (have) {
      const int grow = L.q0 + row;                                     // row within the sequence
      const int r0 = L.q0 + quad * 32;                                 // this warp's first row
      float m_used = -INFINITY, l_run = 0.f;
      const int n_sub = L.n_tiles;
      for (int u = 0; u < n_sub; ++u) {
        const int g = g0 + u;
        const int c0 = u * kAtBN;
        // 32-column chunks of this tile that some row of the warp may see
        const int n_ch = min(4, (min(L.q_hi, r0 + 32) - c0 + 31) >> 5);
        mbar_wait_spin(bar(x, S_FULL), (uint32_t)g & 1u, abort_flag);
        if (lane == 0 && quad < 3 && !*abort_flag) {
          // Q K_u^T and P_{u-1} V_{u-1} have completed: the K slot and (from the second tile on) the V slot are free;
          // behind the item's last Q K^T so is the Q slot, and both go to the next item
          if (u + 1 < n_sub) {
            if (issue_k) load_kv(I, L, u + 1, 0);
          } else if (have_next) {
            if (issue_q) load_q(In, Ln);
            if (issue_k) load_kv(In, Ln, 0, 0);
          }
          if (u > 0 && issue_v) load_kv(I, L, u, 1);
        }
        // Turn-taking between the two warps of a scheduler (this one and the other lane's warp of the same quadrant).
        // Left alone the lanes fall into step: both softmax together (tensor pipe idle), then both MMA blocks
        // together (these warps idle).  A warp that finds its twin inside a softmax pass waits for it to finish, so
        // that the lanes settle half a period apart; lane A has the right of way when both arrive together.  Worth
        // 2-4 % on items of many key tiles, a loss on short ones (the wait is exposed at the item's end), hence the
        // threshold.  The wait is bounded by time and purely a matter of speed.
        const bool take_turns = n_ch >= 2 && n_sub >= kAtTurnTiles;
        if (take_turns && lane == 0) {
          volatile int* mine = in_softmax + 4 * x + quad;
          volatile int* twin = in_softmax + 4 * (x ^ 1) + quad;
          const long long t0 = clock64();
          *mine = 1;
          __threadfence_block();
          if (x == 0) {
            while (*twin && clock64() - t0 < 4000) { }
          } else if (*twin) {
            *mine = 0;
            while (*twin && clock64() - t0 < 4000) { }
            *mine = 1;
          }
        }
        __syncwarp();
        tc_fence_after();
        at_softmax_chunks<1>(s_addr, o_addr, n_ch, grow - c0, c0 - r0, grow < L.q_hi, u > 0, a.scale_log2, m_used, l_run);
        if (take_turns && lane == 0) in_softmax[4 * x + quad] = 0;
        if (u == n_sub - 1 && L.q_hi == I.n) {
          // last tile of the sequence: the P V covers keys up to the next multiple of 16; zero the V rows between
          // the sequence's end and that bound (both 64-dim halves).  Other query tiles need nothing: rows past
          // their end are the sequence's own and P is 0 there.
          const int valid = I.n - u * kAtBN, pad = at_cols(L, u) - valid;
          if (pad > 0) {
            mbar_wait_spin(bar(x, V_FULL), (uint32_t)g & 1u, abort_flag);
            char* v_s = slot(x, 2);
            for (int w = quad * 32 + lane; w < pad * 16; w += 128) {
              const int r = valid + (w >> 4);
              *reinterpret_cast<uint4*>(v_s + ((w >> 3) & 1) * (kAtBN * 128) + r * 128 + (w & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(x, P_FULL));
      }
      // ---- epilogue: O / l -> bf16 -> out[b][row][h][:], 32 columns at a time, two blocks per round through this
      // warp's staging (16-byte units XOR-swizzled by row pair: the 64-byte swizzle of the tensor map)
      const int gl = g0 + n_sub - 1;
      const bool have_next2 = have_next && next_own(In2, Ln2);
      mbar_wait_spin(bar(x, PV_DONE), (uint32_t)gl & 1u, abort_flag);   // MMAs complete in order: all of O is in
      if (issue_v && have_next && !*abort_flag) load_kv(In, Ln, 0, 1);   // and the V slot is free
      __syncwarp();
      tc_fence_after();
      const float inv = 1.0f / l_run;
      const int rows_here = L.q_hi - r0;                               // owned rows among this warp's 32
      const bool whole = rows_here >= 32;                              // warp-uniform
      __nv_bfloat16* otile = a.out + (((size_t)I.b * a.n_max + r0) * a.H + I.h) * 128;
#pragma unroll 1
      for (int rd = 0; rd < 2; ++rd) {                   // not unrolled: once per item, short code counts for more
        uint32_t o[64];
        tmem_ld64(o_addr + rd * 64, o);
        // the stores that read this staging last (the previous round, or the previous item) must have read it
        if (lane == 0) bulk_wait_read<0>();
        tmem_ld_wait();
        if (rd == 1) tc_fence_before();                  // all of O is in registers: the next item may overwrite it
        __syncwarp();
        if (rd == 1 && lane == 0) mbar_arrive(bar(x, O_FREE));
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t* ob = o + 32 * blk + 8 * u;
            uint4 w;
            w.x = cvt_bf16x2(__uint_as_float(ob[0]) * inv, __uint_as_float(ob[1]) * inv);
            w.y = cvt_bf16x2(__uint_as_float(ob[2]) * inv, __uint_as_float(ob[3]) * inv);
            w.z = cvt_bf16x2(__uint_as_float(ob[4]) * inv, __uint_as_float(ob[5]) * inv);
            w.w = cvt_bf16x2(__uint_as_float(ob[6]) * inv, __uint_as_float(ob[7]) * inv);
            *reinterpret_cast<uint4*>(so + blk * 2048 + lane * 64 + ((u ^ ((lane >> 1) & 3)) << 4)) = w;
          }
        }
        if (whole) {
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tma_store_4d(mo, smem_u32(so), rd * 64, I.h, r0, I.b);
            tma_store_4d(mo, smem_u32(so + 2048), rd * 64 + 32, I.h, r0, I.b);
            bulk_commit();
          }
        } else {
          __syncwarp();
#pragma unroll
          for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
            for (int it = 0; it < 4; ++it) {
              const int r = it * 8 + (lane >> 2), u = lane & 3;
              const uint4 w = *reinterpret_cast<const uint4*>(so + blk * 2048 + r * 64 + ((u ^ ((r >> 1) & 3)) << 4));
              if (r < rows_here && DL_IN_BOUNDS(a.status, KID_PREFILL_TC, (((size_t)I.b * a.n_max + r0 + r) * a.H + I.h) * 128 + 127,
                                                (size_t)a.B * a.n_max * a.H * 128))
                *reinterpret_cast<uint4*>(otile + (size_t)r * a.H * 128 + (2 * rd + blk) * 32 + u * 8) = w;
            }
          }
          __syncwarp();                                  // the next round overwrites what these loads read
        }
      }
      g0 += n_sub;
      I = In; L = Ln; have = have_next;
      In = In2; Ln = Ln2; have_next = have_next2;
    }
    if (lane == 0) bulk_wait_read<0>();                  // staged data must be read before shared memory goes
    if (lane == 0 && quad < 3 && *abort_flag) {
      // every copy that was requested must land before the CTA's shared memory is released: per slot at most one is
      // in flight, the last one requested
      for (int w = 0; w < 3; ++w)
        if (issued[w] > 0)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(bar(x, Q_FULL + w), (uint32_t)(issued[w] - 1) & 1u); ++i) __nanosleep(40);
    }
    if (*abort_flag && row == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
  } else {
    // ---------------------------------------------------------------- warp 11: the top rows the lanes leave out
    reg_dec<kAtRegsSmall>();                             // same budget as the rest of its warpgroup (warp 8 idles)
    if (warp == 11) {
      AtWalker W(a);
      AtItem I;
      while (W.next(I, 0)) {
        // the pair's later tile if it is that small, else its earlier one if that is
        const int s = I.q_hi <= kAtTopRows ? I.q_hi : I.q_hi - kAtBM;
        if (s > 0 && s <= kAtTopRows) at_top_rows(a, I, s, lane);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 11) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

bool attn_prefill_tc_supported(const dl_ctx* ctx) {
  const dl_model_desc& d = ctx->desc;
  return d.dtype == DL_BF16 && d.head_dim == 128 && ctx->tmap_encode != nullptr && (size_t)ctx->smem_optin >= kAtSmem;
}

cudaError_t launch_attn_prefill_tc(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                     const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max, float scale,
                                     void* out, cudaStream_t s) {
  if (B == 0 || n_max == 0) return cudaSuccess;
  AtMaps maps;
  AtArgs a;
  long long items = 0;
  cudaError_t e = at_prepare(ctx, q, k_cache, v_cache, cache_len, B, cap, n_max, scale, out, &maps, &a, &items);
  if (e != cudaSuccess) return e;
  static int attr_set[64];
  if (!attr_set[ctx->device & 63]) {
    e = cudaFuncSetAttribute(attn_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmem);
    if (e != cudaSuccess) return e;
    attr_set[ctx->device & 63] = 1;
  }
  const int grid = (int)std::min<long long>(items, (long long)ctx->sm_count);
  attn_prefill_tc_kernel<<<grid, kAtThreads, kAtSmem, s>>>(maps, a);
  return cudaGetLastError();
}

}  // namespace dl
