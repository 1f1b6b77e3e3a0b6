// Prefill attention over the reduced set on the tensor cores (Eq. 1 applied to S^{P*}):
// row i of a sequence's compact context attends rows 0..i of the same context.
// bf16, head_dim 128.  One persistent CTA per SM walks work items (sequence, head, PAIR of 128-row
// query tiles), longest pairs first.  The two query tiles of a pair run as two lanes, A (the later rows)
// and B (the 128 rows before them): each lane has its own Q buffers, its own score / output
// accumulators in tensor memory, its own MMA-issuing thread and its own four softmax warps, and both
// read the same K and V tiles, which are fetched once per pair into a ring shared by the lanes.
// While one lane's softmax warps work on a score tile the tensor pipe runs the other lane's MMAs.
// Pairs are aligned to the END of a sequence (rows [n-256(p+1), n-256p)), so the ragged pair is the
// one at the top of the causal triangle, where it needs the fewest keys; lane B of a pair that has
// 128 rows or fewer does not exist and the lane moves on to the next item on its own.
//   warp 8     : TMA producer (one lane), a polling loop over three cursors: the K/V ring (tiles of
//                128 keys, K and V alternating, three slots of 32 KB) and the Q loads of either lane
//                (two slots per lane, so an item's Q is in flight while the previous item computes).
//   warps 9,10 : the MMA-issuing thread of lane A / lane B:
//                S = Q K^T (128 x N, K-major operands from shared memory), O += P V (P read from
//                tensor memory, V as an MN-major shared-memory operand), then the next tile's Q K^T;
//                completion signals follow the block, the softmax's first.
//                Full tiles use N = 128 keys; a lane's last tile uses N = keys left rounded up to 16,
//                in both products, so the tensor pipe does not multiply by padding.
//   warps 0-3 / 4-7 : softmax of lane A / B, one query row per thread, straight out of tensor memory
//                in one pass of 32-column chunks (the next chunk's load in flight meanwhile; these warps
//                take the registers the other warps give back).  Chunks that no row of the warp may see
//                (above the causal diagonal) are skipped.  The running maximum is only raised when the
//                tile's maximum exceeds it by more than 2^8 (then O is rescaled in tensor memory and the
//                tile redone), so most tiles never touch O.  P (bf16) overwrites the first half of S.  The same warps
//                normalise O and write the output: 32 x 32 blocks staged in the item's own Q buffer
//                (free once its last Q K^T has run) and sent with TMA stores; a clipped tile at the
//                top of a sequence, whose surplus rows belong to the next tile, is written with
//                predicated stores instead.  The Q slot returns to the producer once those stores
//                have read it.
//   warp 11    : tensor-memory allocation (all 512 columns: O_A | S_A | O_B | S_B); then the top rows of sequences
//                whose length leaves a top tile of at most 16 rows (attn_prefill_top.cuh), which the lanes skip.
// Barrier phases are driven by running counters (ring tiles, a lane's tiles, a lane's items) that every
// role advances identically.  Rows past a sequence's length are fetched with the tile (they are
// masked); where the 16-row rounding of the last tile reaches past the sequence's end, those V rows
// are zeroed in shared memory first, since 0 * x must stay 0 for any bit pattern.  Every wait is
// bounded (pipeline.cuh); an abort leaves DL_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

#include "attn_prefill.cuh"
#include "attn_prefill_softmax.cuh"
#include "attn_prefill_top.cuh"

namespace dl {


__global__ void __launch_bounds__(kAtThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ AtMaps maps, const AtArgs a) {
  extern __shared__ __align__(1024) char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (smem_u32(smem) & 1023u) {                        // the swizzled tiles need 1024-byte alignment
    if (tid == 0) report_status(a.status, DL_ERR_ALIGNMENT, -1);
    return;
  }
  char* ring_s = smem + kAtOffRing;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAtOffBar);
  // Ring tile T of this CTA (running count over its items; K and V of key tile j of an item are tiles
  // base + 2j and base + 2j + 1) lives in slot T % 3 and completes phase (T / 3) & 1 of that slot's
  // `full` barrier; lane X's MMAs that read it complete a phase of the slot's `free_X` barrier.
  // A lane's own barriers: its g-th key tile (running count) completes phase g & 1 of s_full / p_full /
  // pv_done (a waiter is never two phases behind: before tile g's S is ready, the P V of g - 1 has
  // completed); its i-th item completes
  // phase i & 1 of o_free and phase (i >> 1) & 1 of q_full / q_done of Q slot i & 1.
  auto ring_full = [&](int s) { return smem_u32(bars + s); };
  auto ring_free = [&](int x, int s) { return smem_u32(bars + 3 + 3 * x + s); };
  auto q_full = [&](int x, int s) { return smem_u32(bars + 9 + 2 * x + s); };    // Q tile has landed
  auto q_done = [&](int x, int s) { return smem_u32(bars + 13 + 2 * x + s); };   // Q slot may be refilled (4 warps)
  auto s_full = [&](int x, int b) { return smem_u32(bars + 17 + 2 * x + b); };   // Q K^T has completed: S ready
  auto p_full = [&](int x, int b) { return smem_u32(bars + 21 + 2 * x + b); };   // P is in tensor memory (4 warps)
  auto pv_done = [&](int x, int b) { return smem_u32(bars + 25 + 2 * x + b); };  // P V has completed: O at rest
  auto o_free = [&](int x) { return smem_u32(bars + 29 + x); };   // the epilogue has read O (4 warps)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 33);

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kAtRing; ++s) {
      mbar_init(ring_full(s), 1);
      mbar_init(ring_free(0, s), 1);
      mbar_init(ring_free(1, s), 1);
    }
    for (int x = 0; x < 2; ++x) {
      for (int s = 0; s < 2; ++s) { mbar_init(q_full(x, s), 1); mbar_init(q_done(x, s), 4); }
      for (int b = 0; b < 2; ++b) {
        mbar_init(s_full(x, b), 1);
        mbar_init(p_full(x, b), 4);
        mbar_init(pv_done(x, b), 1);
      }
      mbar_init(o_free(x), 4);
    }
    fence_mbar_init();
  }
  if (warp == 11) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 8) {
    // ---------------------------------------------------------------- TMA producer
    reg_dec<kAtRegsSmall>();
    if (lane == 0) {
      for (int i = 0; i < 4; ++i) {
        tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(maps.q[i]));
        tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(maps.k[i]));
        tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(maps.v[i]));
      }
      // Two cursors over the CTA's items: the ring's (K and V tiles, in order) and the Q loads' (per item, either
      // lane's tile as soon as its slot is free; the item is left when both are on their way).  Each cursor
      // advances in ONE place: the walker's step is inlined wherever it is called, and this role's code is
      // fetched cold at every item.
      AtWalker Wr(a), Wq(a);
      AtItem Ir, Iq;
      int T = 0, jr = 0;                       // ring tiles issued so far / tile index within Ir (K, V alternating)
      int nq[2] = {0, 0};                      // Q loads issued so far per lane
      bool hr = true, hq = true, need_r = true, need_q = true;
      int q_todo = 0;                          // lanes of Iq whose Q tile is still to be requested (bit x)
      int idle = 0;
      while ((hr || hq) && !*abort_flag) {
        bool prog = false;
        if (hq && need_q) {
          hq = Wq.next(Iq, kAtTopRows);
          need_q = false;
          q_todo = hq ? ((at_lane(Iq, 0).exists ? 1 : 0) | (at_lane(Iq, 1).exists ? 2 : 0)) : 0;
          prog = true;
        }
#pragma unroll 1
        for (int x = 0; x < 2; ++x) {
          if (!((q_todo >> x) & 1)) continue;
          const int s = nq[x] & 1;
          // the slot's previous item (two items back) must have finished its epilogue
          if (nq[x] >= 2 && !mbar_test(q_done(x, s), ((nq[x] - 2) >> 1) & 1)) continue;
          const AtLane L = at_lane(Iq, x);
          char* dst = smem + (2 * x + s) * kAtTile;
          // the rows the lane owns, in 16s (a tile clipped at the top of the sequence owns fewer than 128)
          const int bx = at_box(min(kAtBM, (L.q_hi - L.q0 + 15) & ~15));
          const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(maps.q[bx]);
          mbar_expect_tx(q_full(x, s), kAtTile >> bx);
          tma_load_2d(smem_u32(dst), mq, 0, Iq.row_base + L.q0, q_full(x, s));
          tma_load_2d(smem_u32(dst + kAtBM * 128), mq, 64, Iq.row_base + L.q0, q_full(x, s));
          ++nq[x];
          q_todo &= ~(1 << x);
          prog = true;
        }
        if (hq && !need_q && q_todo == 0) need_q = true;
        if (hr && need_r) {
          hr = Wr.next(Ir, kAtTopRows);
          need_r = false;
          jr = 0;
          prog = true;
        }
        if (hr && !need_r) {
          const int s = T % kAtRing;
          bool slot_free = true;
          if (T >= kAtRing) {
            // both lanes have released the slot's previous tile (a lane releases every tile, read or not)
            const uint32_t par = (uint32_t)(T / kAtRing - 1) & 1u;
            slot_free = mbar_test(ring_free(0, s), par) && mbar_test(ring_free(1, s), par);
          }
          if (slot_free) {
            const int j = jr >> 1;
            char* dst = ring_s + s * kAtTile;
            // keys of the tile that the pair's later query tile covers (the earlier one never needs more)
            const int bx = at_box(min(kAtBN, (Ir.q_hi - j * kAtBN + 15) & ~15));
            const CUtensorMap* m = reinterpret_cast<const CUtensorMap*>((jr & 1) ? maps.v[bx] : maps.k[bx]);
            const int r = Ir.row_base + j * kAtBN;
            mbar_expect_tx(ring_full(s), kAtTile >> bx);
            tma_load_2d(smem_u32(dst), m, 0, r, ring_full(s));
            tma_load_2d(smem_u32(dst + kAtBN * 128), m, 64, r, ring_full(s));
            ++T;
            if (++jr == 2 * Ir.n_kv) need_r = true;
            prog = true;
          }
        }
        if (prog) {
          idle = 0;
        } else if (++idle > kSpinLimitBusy) {
          *abort_flag = 1;
        }
      }
      if (*abort_flag) {
        // every copy that was issued must land before the CTA's shared memory is released
        report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
        for (int t = max(0, T - kAtRing); t < T; ++t)
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(ring_full(t % kAtRing), (t / kAtRing) & 1); ++i) __nanosleep(40);
        for (int x = 0; x < 2; ++x)
          for (int t = max(0, nq[x] - 2); t < nq[x]; ++t)
            for (int i = 0; i < kSpinLimit && !mbar_try_wait(q_full(x, t & 1), (t >> 1) & 1); ++i) __nanosleep(40);
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ---------------------------------------------------------------- MMA issuer of one lane
    reg_dec<kAtRegsSmall>();
    if (lane == 0) {
      const int x = warp - 9;
      const uint32_t t_o = tmem + x * kAtLaneCols + kAtColO, t_s = tmem + x * kAtLaneCols + kAtColS;
      const uint32_t idesc_pv = idesc_bf16(kAtBM, 128, 0, 1);          // B (= V) is MN-major
      AtWalker W(a);
      AtItem I;
      int n_item = 0, g0 = 0, T0 = 0;                 // this lane's items / tiles so far; ring tiles before this item
      while (W.next(I, kAtTopRows)) {
        const AtLane L = at_lane(I, x);
        auto wait_ring = [&](int T) { mbar_wait_spin(ring_full(T % kAtRing), (T / kAtRing) & 1, abort_flag); };
        const int n_sub = L.exists ? L.n_tiles : 0;
        const int qs = n_item & 1;
        const uint64_t q_desc = smem_desc_sw128(smem_u32(smem + (2 * x + qs) * kAtTile));
        // Block u of the item: O += P_u V_u, then S = Q K_{u+1}^T (which overwrites P: in order behind the P V).
        // Block -1 is the first Q K^T alone, the last block the last P V alone.  One copy of the code for all
        // of them, loops not unrolled: an MMA holds the thread for 64 cycles anyway, and this role's code is
        // fetched cold at every item.
        for (int u = L.exists ? -1 : 0; u < n_sub; ++u) {
          const int g = g0 + u;
          const int Tv = T0 + 2 * u + 1, sv = Tv % kAtRing;              // the V tile of this key tile
          const int sk = (Tv + 1) % kAtRing;                             // the K tile of the next one
          const bool has_pv = u >= 0, has_qk = u + 1 < n_sub;
          // operands first (they land long before), then the softmax's hand-over
          if (has_pv) wait_ring(Tv);
          else mbar_wait_spin(q_full(x, qs), (n_item >> 1) & 1, abort_flag);
          if (has_qk) wait_ring(Tv + 1);
          if (u == 0) mbar_wait_spin(o_free(x), (n_item & 1) ^ 1, abort_flag);   // previous item's O has been read
          if (has_pv) {
            // polled without suspending: the wake-up of a suspended wait costs this thread ~600 cycles per tile
            const uint32_t pb = p_full(x, 0), ph = (uint32_t)g & 1u;
            int spins = 0;
            while (!mbar_test(pb, ph)) {
              if ((++spins & 1023) == 0 && (*abort_flag || spins > (kSpinLimitBusy << 4))) { *abort_flag = 1; break; }
            }
          }
          tc_fence_after();
          if (has_pv) {
            uint64_t v_desc = smem_desc_sw128_mn(smem_u32(ring_s + sv * kAtTile), kAtBN * 128);
            const int ksteps = at_cols(L, u) >> 4;
#pragma unroll 1
            for (int ks = 0; ks < ksteps; ++ks, v_desc += 2048 >> 4)
              mma_ts(t_o, t_s + ks * 8, v_desc, idesc_pv, (u | ks) != 0);
          }
          if (has_qk) {
            // 16 dims further per step, and from the fourth step on in the tile's second 64-dim half
            uint64_t qd = q_desc, kd = smem_desc_sw128(smem_u32(ring_s + sk * kAtTile));
            const uint32_t idesc_qk = idesc_bf16(kAtBM, (uint32_t)at_cols(L, u + 1));
#pragma unroll 1
            for (int ks = 0; ks < 8; ++ks) {
              mma_ss(t_s, qd, kd, idesc_qk, ks != 0);
              const uint64_t step = (ks == 3) ? (uint64_t)((kAtBM * 128 - 96) >> 4) : 2ull;
              qd += step;
              kd += step;
            }
            // Completion signals: a commit covers every MMA this thread has issued so far.
            mma_commit(s_full(x, 0));                                    // first: the softmax warps wait on it
            mma_commit(ring_free(x, sk));
          }
          if (has_pv) {
            mma_commit(pv_done(x, 0));
            mma_commit(ring_free(x, sv));
          }
        }
        // A lane does not read every ring tile (not the pair's last key tile when it has the earlier query
        // tile, nothing of a pair that has no earlier tile).  It still observes every tile's landing and
        // releases it, in ring order, so that the slot barriers advance one phase per tile for every
        // waiter: a waiter that had skipped phases could not tell them apart by parity.
        for (int T = T0 + 2 * n_sub; T < T0 + 2 * I.n_kv; ++T) {
          wait_ring(T);
          mbar_arrive(ring_free(x, T % kAtRing));
        }
        if (L.exists) {
          g0 += n_sub;
          ++n_item;
        }
        T0 += 2 * I.n_kv;
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
    AtWalker W(a);
    AtItem I;
    int n_item = 0, g0 = 0, T0 = 0;
    int q_slot_held = -1;                                              // Q slot whose staged stores are still in flight
    while (W.next(I, kAtTopRows)) {
      const AtLane L = at_lane(I, x);
      if (!L.exists) { T0 += 2 * I.n_kv; continue; }
      const int grow = L.q0 + row;                                     // row within the sequence
      const int r0 = L.q0 + quad * 32;                                 // this warp's first row
      float m_used = -INFINITY, l_run = 0.f;
      const int n_sub = L.n_tiles;
      for (int u = 0; u < n_sub; ++u) {
        const int g = g0 + u, sbuf = 0;
        const int c0 = u * kAtBN;
        const uint32_t sa = s_addr;
        // 32-column chunks of this sub-tile that some row of the warp may see
        const int n_ch = min(4, (min(L.q_hi, r0 + 32) - c0 + 31) >> 5);
        mbar_wait_spin(s_full(x, sbuf), g & 1, abort_flag);
        tc_fence_after();
        at_softmax_halves<1>(sa, o_addr, n_ch, grow - c0, c0 - r0, grow < L.q_hi, u > 0, a.scale_log2, m_used, l_run);
        if (u == n_sub - 1 && L.q_hi == I.n) {
          // last tile of the sequence (only lane A of pair 0 gets here): the P V covers keys up to the next
          // multiple of 16; zero the V rows between the sequence's end and that bound (both 64-dim halves).
          // Other query tiles need nothing: rows past their end are the sequence's own and P is 0 there.
          const int j = u;
          const int valid = I.n - j * kAtBN, pad = at_cols(L, j) - valid;
          if (pad > 0) {
            const int T = T0 + 2 * j + 1, s = T % kAtRing;
            mbar_wait_spin(ring_full(s), (T / kAtRing) & 1, abort_flag);
            char* v_s = ring_s + s * kAtTile;
            for (int u = quad * 32 + lane; u < pad * 16; u += 128) {
              const int r = valid + (u >> 4);
              *reinterpret_cast<uint4*>(v_s + ((u >> 3) & 1) * (kAtBN * 128) + r * 128 + (u & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full(x, sbuf));
        if (q_slot_held >= 0) {
          // the previous item's staged output has long been read: hand its Q slot back to the producer
          if (lane == 0) { bulk_wait_read<0>(); mbar_arrive(q_done(x, q_slot_held)); }
          q_slot_held = -1;
        }
      }
      // ---- epilogue: O / l -> bf16 -> out[b][row][h][:], 32 columns at a time, staged in this warp's 8 KB of
      // the item's Q slot (16-byte units XOR-swizzled by row pair: the 64-byte swizzle of the tensor map)
      const int gl = g0 + n_sub - 1;
      mbar_wait_spin(pv_done(x, 0), gl & 1, abort_flag);   // MMAs complete in order: all of O is in
      tc_fence_after();
      const float inv = 1.0f / l_run;
      const int rows_here = L.q_hi - r0;                               // owned rows among this warp's 32
      const bool whole = rows_here >= 32;                              // warp-uniform
      const int qs = n_item & 1;
      char* so = smem + (2 * x + qs) * kAtTile + quad * 8192;
      __nv_bfloat16* otile = a.out + (((size_t)I.b * a.n_max + r0) * a.H + I.h) * 128;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {                   // not unrolled: once per item, short code counts for more
        uint32_t o[32];
        tmem_ld32(o_addr + cc * 32, o);
        tmem_ld_wait();
        if (cc == 3) {                                   // all of O is in registers: the next item may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(o_free(x));
        }
        char* sb = so + cc * 2048;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          uint4 w;
          w.x = cvt_bf16x2(__uint_as_float(o[8 * u]) * inv, __uint_as_float(o[8 * u + 1]) * inv);
          w.y = cvt_bf16x2(__uint_as_float(o[8 * u + 2]) * inv, __uint_as_float(o[8 * u + 3]) * inv);
          w.z = cvt_bf16x2(__uint_as_float(o[8 * u + 4]) * inv, __uint_as_float(o[8 * u + 5]) * inv);
          w.w = cvt_bf16x2(__uint_as_float(o[8 * u + 6]) * inv, __uint_as_float(o[8 * u + 7]) * inv);
          *reinterpret_cast<uint4*>(sb + lane * 64 + ((u ^ ((lane >> 1) & 3)) << 4)) = w;
        }
      }
      if (whole) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) tma_store_4d(mo, smem_u32(so + cc * 2048), cc * 32, I.h, r0, I.b);
        }
      } else {
        __syncwarp();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
          for (int it = 0; it < 4; ++it) {
            const int r = it * 8 + (lane >> 2), u = lane & 3;
            const uint4 w = *reinterpret_cast<const uint4*>(so + cc * 2048 + r * 64 + ((u ^ ((r >> 1) & 3)) << 4));
            if (r < rows_here) *reinterpret_cast<uint4*>(otile + (size_t)r * a.H * 128 + cc * 32 + u * 8) = w;
          }
        }
      }
      if (lane == 0) bulk_commit();
      __syncwarp();
      q_slot_held = qs;
      g0 += n_sub;
      ++n_item;
      T0 += 2 * I.n_kv;
    }
    if (q_slot_held >= 0 && lane == 0) { bulk_wait_read<0>(); mbar_arrive(q_done(x, q_slot_held)); }
    if (*abort_flag && row == 0) report_status(a.status, DL_ERR_TIMEOUT, blockIdx.x);
  } else {
    // ---------------------------------------------------------------- warp 11: the top rows the lanes leave out
    reg_dec<kAtRegsSmall>();                             // same budget as the rest of its warpgroup
    AtWalker W(a);
    AtItem I;
    while (W.next(I, 0)) {
      // the pair's later tile if it is that small, else its earlier one if that is
      const int s = I.q_hi <= kAtTopRows ? I.q_hi : I.q_hi - kAtBM;
      if (s > 0 && s <= kAtTopRows) at_top_rows(a, I, s, lane);
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
