// Top-k vision-token selection (TopkArgmax_k of Eq. 11) and the decode keep test (Eq. 5 / 6).
//
// One CTA per sequence.  Scores become order-preserving 32-bit keys (after -0 -> +0 and
// NaN -> -inf), a 4-pass 8-bit radix select finds the k-th largest key T and how many keys
// equal to T still belong to the selection, and two ordered block scans turn that into the
// 0/1 mask and the ascending index list.  Between equal scores the lower index wins, so the
// result is unique and reproducible bit for bit.
#include "common.cuh"

namespace dl {

constexpr int kTopkThreads = 512;

__device__ __forceinline__ uint32_t score_key(float s, bool* was_nan) {
  uint32_t u = __float_as_uint(s);
  if ((u & 0x7fffffffu) > 0x7f800000u) { *was_nan = true; u = 0xff800000u; }  // NaN -> -inf
  if (u == 0x80000000u) u = 0u;                                                // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive block scan of one int per thread, in thread order; returns the exclusive prefix
// and leaves the block total in *total.  `warp_sums` has kTopkThreads/32 ints.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = (lane < kTopkThreads / 32) ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    if (lane < kTopkThreads / 32) warp_sums[lane] = wi - w;   // exclusive warp offsets
    if (lane == kTopkThreads / 32 - 1) *total = wi;
  }
  __syncthreads();
  int res = warp_sums[warp] + incl - v;
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ score, const int32_t* __restrict__ n_vis,
            const int32_t* __restrict__ k_arr, int32_t n_max, int32_t* __restrict__ kept_idx,
            int32_t k_max, uint8_t* __restrict__ keep, DeviceStatus* st) {
  extern __shared__ uint32_t keys[];          // [n_max]
  __shared__ int hist[256];
  __shared__ int warp_sums[kTopkThreads / 32];
  __shared__ int sh_total;
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;

  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  int n = n_vis ? n_vis[b] : n_max;
  n = max(0, min(n, n_max));
  int kk = max(0, min(k_arr[b], n));
  const float* s = score + (size_t)b * n_max;

  bool saw_nan = false;
  for (int i = tid; i < n; i += kTopkThreads) keys[i] = score_key(s[i], &saw_nan);
  if (saw_nan) report_status(st, DL_WARN_NAN, b);
  if (tid == 0 && kept_idx != nullptr && kk > k_max) report_status(st, DL_ERR_INVALID_ARG, b);   // the index list is cut
  if (tid == 0) { sh_prefix = 0u; sh_remaining = kk; }
  __syncthreads();

  // ---- radix select: after the loop sh_prefix is the kk-th largest key and sh_remaining
  //      the number of keys equal to it that are selected (lowest indices first)
  uint32_t mask = 0u;
  if (kk > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = tid; i < 256; i += kTopkThreads) hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = sh_prefix;
      for (int i = tid; i < n; i += kTopkThreads) {
        uint32_t key = keys[i];
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xff], 1);
      }
      __syncthreads();
      if (tid < 32) {
        // the digit d with (keys in higher digits) < remaining <= (keys in digits >= d), found by one warp:
        // lane l owns the eight digits 255 - 8l .. 248 - 8l, highest first
        const int rem = sh_remaining;
        int c[8], lane_total = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = hist[255 - 8 * tid - j]; lane_total += c[j]; }
        int incl = lane_total;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += v;
        }
        int above = incl - lane_total;                       // keys in the digits of lower lanes (higher digits)
        const bool mine = above < rem && rem <= incl;
        const unsigned who = __ballot_sync(0xffffffffu, mine);
        if (who == 0u) {
          // fewer keys than asked for cannot happen (remaining <= keys under the prefix); digit 0 as a guard
          if (tid == 31) { sh_remaining = max(1, rem - (incl - c[7])); sh_prefix = prefix; }
        } else if (mine) {
          int d = 255 - 8 * tid, r = rem - above;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (c[j] >= r) break;
            r -= c[j];
            --d;
          }
          sh_remaining = r;
          sh_prefix = prefix | ((uint32_t)d << shift);
        }
      }
      mask |= 0xffu << shift;
      __syncthreads();
    }
  }
  const uint32_t T = sh_prefix;
  const int take_eq = sh_remaining;

  // ---- ordered scans over a blocked arrangement: thread t owns items [t*ipt, (t+1)*ipt)
  const int ipt = (n_max + kTopkThreads - 1) / kTopkThreads;
  const int i0 = tid * ipt, i1 = min(n, i0 + ipt);
  int eq_cnt = 0;
  if (kk > 0) for (int i = i0; i < i1; ++i) eq_cnt += (keys[i] == T);
  int eq_rank = block_exclusive_scan(eq_cnt, warp_sums, &sh_total);

  int kept_cnt = 0;
  if (kk > 0) {
    int r = eq_rank;
    for (int i = i0; i < i1; ++i) {
      uint32_t key = keys[i];
      bool kp = key > T;
      if (key == T) { kp = r < take_eq; ++r; }
      kept_cnt += kp;
      keys[i] = kp ? 1u : 0u;                 // reuse the key slot as the flag
    }
  }
  int out_pos = block_exclusive_scan(kept_cnt, warp_sums, &sh_total);

  uint8_t* kp_out = keep + (size_t)b * n_max;
  for (int i = i0; i < min(n_max, i0 + ipt); ++i) {
    bool kp = (kk > 0) && (i < n) && (keys[i] != 0u);
    if (DL_IN_BOUNDS(st, KID_TOPK, (size_t)b * n_max + i, (size_t)gridDim.x * n_max)) kp_out[i] = kp ? 1 : 0;
    if (kp && kept_idx && out_pos < k_max &&
        DL_IN_BOUNDS(st, KID_TOPK, (size_t)b * k_max + out_pos, (size_t)gridDim.x * k_max))
      kept_idx[(size_t)b * k_max + out_pos] = i;
    out_pos += kp;
  }
  if (kept_idx)
    for (int j = kk + tid; j < k_max; j += kTopkThreads) kept_idx[(size_t)b * k_max + j] = -1;
}

cudaError_t launch_topk(const float* score, const int32_t* n_vis, const int32_t* k, int32_t B,
                        int32_t n_vis_max, int32_t* kept_idx, int32_t k_max, uint8_t* keep,
                        DeviceStatus* st, cudaStream_t s) {
  if (B == 0 || n_vis_max == 0) return cudaSuccess;
  size_t smem = (size_t)n_vis_max * sizeof(uint32_t);
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  topk_kernel<<<B, kTopkThreads, smem, s>>>(score, n_vis, k, n_vis_max, kept_idx, k_max, keep, st);
  return cudaGetLastError();
}

// keep[b] = logit[b] > threshold, strictly; NaN compares false and is reported.
__global__ void decode_keep_kernel(const float* __restrict__ logit, int32_t B, float threshold,
                                   uint8_t* __restrict__ keep, DeviceStatus* st) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  float z = logit[b];
  if (z != z) report_status(st, DL_WARN_NAN, b);
  keep[b] = (z > threshold) ? 1 : 0;
}

// Decoding without KV cache (Eq. 12): the mask of all generated tokens of every sequence at once,
// keep iff logit > threshold, with the last valid token of each sequence always kept.
__global__ void nocache_mask_kernel(const float* __restrict__ logit, const int32_t* __restrict__ n_gen,
                                    int32_t B, int32_t n_max, float threshold, uint8_t* __restrict__ keep,
                                    DeviceStatus* st) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_max) return;
  const int n = min(max(n_gen ? n_gen[b] : n_max, 0), n_max);
  uint8_t k = 0;
  if (i < n) {
    const float z = logit[(size_t)b * n_max + i];
    if (z != z) report_status(st, DL_WARN_NAN, (long long)b * n_max + i);
    k = (z > threshold || i == n - 1) ? 1 : 0;
  }
  keep[(size_t)b * n_max + i] = k;
}

cudaError_t launch_nocache_mask(const float* logit, const int32_t* n_gen, int32_t B, int32_t n_max,
                                float threshold, uint8_t* keep, DeviceStatus* st, cudaStream_t s) {
  if (B == 0 || n_max == 0) return cudaSuccess;
  dim3 grid((n_max + 255) / 256, B);
  nocache_mask_kernel<<<grid, 256, 0, s>>>(logit, n_gen, B, n_max, threshold, keep, st);
  return cudaGetLastError();
}

cudaError_t launch_decode_keep(const float* logit, int32_t B, float threshold, uint8_t* keep,
                               DeviceStatus* st, cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  decode_keep_kernel<<<(B + 127) / 128, 128, 0, s>>>(logit, B, threshold, keep, st);
  return cudaGetLastError();
}

}  // namespace dl
