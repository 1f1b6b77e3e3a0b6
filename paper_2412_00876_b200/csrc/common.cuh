// Shared declarations of the library's translation units: context, workspace layout,
// device status word, small device helpers and the kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/dl.h"

namespace dl {

// ---------------------------------------------------------------------------------------
// Device status word (first bytes of the workspace).  Kernels record the FIRST error they
// see with an atomic compare-and-swap on `code`; warnings never overwrite errors.
// ---------------------------------------------------------------------------------------
struct DeviceStatus {
  int32_t code;
  int32_t pad;
  unsigned long long detail;
};

__device__ __forceinline__ void report_status(DeviceStatus* st, int32_t code, long long detail) {
  if (st == nullptr) return;
  int32_t old = atomicCAS(&st->code, 0, code);
  if (old == 0) {
    atomicExch(&st->detail, (unsigned long long)detail);
  } else if (old > 0 && code < 0) {  // an error replaces a warning
    if (atomicCAS(&st->code, old, code) == old) atomicExch(&st->detail, (unsigned long long)detail);
  }
}

// Checked build (-DDL_BOUNDS=1): DL_IN_BOUNDS(status, kernel id, index, extent) is false for an index outside
// [0, extent) and records it; the caller skips the access.  In the normal build it is the constant true.
enum KernelId : int {
  KID_DECODE_MMA = 1, KID_DECODE_SIMT = 2, KID_DECODE_FP8 = 3, KID_COMPACT_PLAN = 4, KID_COMPACT_COPY = 5,
  KID_TOPK = 6, KID_KEEP = 7, KID_PREFILL_TOP = 8, KID_PREFILL_SIMT = 9, KID_PREFILL_TC = 10, KID_QUANTIZE = 11,
  KID_PREDICTOR = 12, KID_SELFTEST = 0x7e
};
#ifdef DL_BOUNDS
__device__ __forceinline__ bool bounds_ok(DeviceStatus* st, int kid, long long idx, long long extent) {
  if (idx >= 0 && idx < extent) return true;
  report_status(st, DL_ERR_BOUNDS, ((long long)kid << 48) | (idx & 0xFFFFFFFFFFFFll));
  return false;
}
#define DL_IN_BOUNDS(st, kid, idx, extent) dl::bounds_ok((st), (kid), (long long)(idx), (long long)(extent))
#else
#define DL_IN_BOUNDS(st, kid, idx, extent) true
#endif

// ---------------------------------------------------------------------------------------
// Workspace layout (all offsets 256-byte aligned).
// ---------------------------------------------------------------------------------------
constexpr int kDecodeMinChunk = 64;   // smallest rows-per-item the decode kernel may be asked for
constexpr int kDecodeScratchSets = 3; // decode scratch sets (see Workspace)
constexpr int kPredMaxSplit = 80;     // most unit tiles of the predictor's hidden layer
constexpr int kPredKSplit = 8;        // most ranges of the hidden dimension a unit tile of the decode-shape predictor is cut into
constexpr int kPredRowTile = 128;     // rows per predictor row tile (tensor-core kernel)

struct Workspace {
  char* base = nullptr;
  int64_t bytes = 0;
  int32_t max_batch = 0, max_rows = 0, cap = 0;
  // sub-buffers
  DeviceStatus* status = nullptr;
  int32_t* plan_base = nullptr;       // [max_batch] compaction: first destination row
  int32_t* plan_count = nullptr;      // [max_batch] compaction: rows to append (-1: skip sequence)
  // decode scratch, three sets: up to three consecutive layers of a stack are in flight at a time
  int32_t* dec_ticket = nullptr;      // [3][max_batch * H] arrivals per (b,h); zero between launches
  float* dec_partial = nullptr;       // [3][max_batch * H * dec_slots * (D + 2)]
  int32_t dec_slots = 0;              // partial slots per (b,h)
  int32_t* dec_commit = nullptr;      // [2] CTAs of a committing attention launch that have finished (slot 0: compact
                                      // layers, slot 1: dense layers); zero between launches
  uint8_t* ones = nullptr;            // [max_batch] the keep-all decision of dense layers
  float* pred_partial = nullptr;      // [kPredMaxSplit][max_rows padded to kPredRowTile]
  int32_t* pred_ticket = nullptr;     // [row tiles]; zero between launches
  float* pred_split = nullptr;        // [unit tiles][kPredKSplit][kPredRowTile][tile width] raw sums of the decode-shape predictor
  int32_t* pred_split_ticket = nullptr;   // [kPredMaxSplit]; zero between launches
  int32_t pred_rows_padded = 0;
};

int64_t workspace_layout(const dl_model_desc& d, int32_t max_batch, int32_t max_rows, int32_t cap,
                         Workspace* ws /* may be null: size query only */);

struct Options {
  int32_t predictor_impl = 0;
  int32_t prefill_attn_impl = 0;
  int32_t decode_chunk = 0;
  int32_t decode_impl = 0;
  int32_t compact_impl = 0;            // 0 auto, 1 register-staged copy kernel, 2 bulk-copy (TMA) kernel
  int32_t in_layer_stack = 0;          // set by the layer-stack call around its launches (not a user option)
};

}  // namespace dl

struct dl_ctx {
  int32_t device = 0;
  dl_model_desc desc{};
  dl::Workspace ws{};
  dl::Options opt{};
  int32_t sm_count = 0;
  int32_t smem_optin = 0;
  cudaError_t last_cuda = cudaSuccess;
  void* tmap_encode = nullptr;        // cuTensorMapEncodeTiled, resolved at create
  // copy streams and events of the pipelined host-fed decode (dl_decode_steps_host), created on first use
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  cudaEvent_t ev_fork = nullptr;
  // tensor maps of cache tensors seen before (decode attention); see attn_decode.cu
  static constexpr int kMapCache = 256;
  struct MapEntry { const void* base = nullptr; long long rows = 0, aux = 0; unsigned char map[128]; };
  mutable MapEntry map_cache[kMapCache];
  mutable int map_next = 0;
};

namespace dl {

// ---------------------------------------------------------------------------------------
// element helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// exact-erf GELU in fp32
__device__ __forceinline__ float gelu_erf(float h) { return 0.5f * h * (1.0f + erff(h * 0.70710678118654752440f)); }

// ---------------------------------------------------------------------------------------
// kernel launchers (one per translation unit); all return the launch's cudaError_t
// ---------------------------------------------------------------------------------------
cudaError_t launch_topk(const float* score, const int32_t* n_vis, const int32_t* k, int32_t B,
                        int32_t n_vis_max, int32_t* kept_idx, int32_t k_max, uint8_t* keep,
                        DeviceStatus* st, cudaStream_t s);

cudaError_t launch_compact(const dl_ctx* ctx, const void* k_src, const void* v_src, const uint8_t* keep,
                           int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                           void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, cudaStream_t s,
                           int32_t force_impl = 0, int32_t reuse_plan = 0, int32_t chained = 0);

cudaError_t launch_commit_len(const uint8_t* keep, int32_t B, int32_t cap, int32_t* cache_len,
                              cudaStream_t s);

cudaError_t launch_attn_decode(const dl_ctx* ctx, const void* q, const void* k_t, const void* v_t,
                               void* k_cache, void* v_cache, const int32_t* cache_len,
                               const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                               bool overlap_prev, int scratch_set, cudaStream_t s, int32_t* commit_len = nullptr,
                               int commit_slot = 0);

cudaError_t launch_quantize_kv_fp8(const dl_ctx* ctx, const void* src, const int32_t* cache_len, const float* scale,
                                   int32_t B, int32_t cap, void* dst, cudaStream_t s);
cudaError_t launch_attn_decode_fp8(const dl_ctx* ctx, const void* q, const void* k_t, const void* v_t, void* k_cache,
                                   void* v_cache, const float* k_scale, const float* v_scale, const int32_t* cache_len,
                                   const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                                   cudaStream_t s, bool in_stack = false, bool overlap_prev = false, int scratch_set = 0);

cudaError_t launch_predictor_simt(const dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows,
                                  float* score, cudaStream_t s);
// keep != nullptr: also keep[r] = score[r] > threshold (the decode decision, taken where the score is completed)
cudaError_t launch_predictor_tc(dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows,
                                float* score, cudaStream_t s, uint8_t* keep = nullptr, float threshold = 0.f);
bool predictor_tc_supported(const dl_ctx* ctx);

cudaError_t launch_decode_keep(const float* logit, int32_t B, float threshold, uint8_t* keep,
                               DeviceStatus* st, cudaStream_t s);

cudaError_t launch_nocache_mask(const float* logit, const int32_t* n_gen, int32_t B, int32_t n_max,
                                float threshold, uint8_t* keep, DeviceStatus* st, cudaStream_t s);

cudaError_t launch_attn_prefill_simt(const dl_ctx* ctx, const void* q, const void* k_cache,
                                     const void* v_cache, const int32_t* cache_len, int32_t B,
                                     int32_t cap, int32_t n_max, float scale, void* out, cudaStream_t s);
cudaError_t launch_attn_prefill_tc(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max,
                                   float scale, void* out, cudaStream_t s);
bool attn_prefill_tc_supported(const dl_ctx* ctx);

int64_t predictor_paper_scratch_bytes(int64_t rows);
bool predictor_paper_supported(const dl_ctx* ctx);
cudaError_t launch_predictor_paper(dl_ctx* ctx, const dl_predictor2* p, const void* x, const int32_t* n_vis, int32_t B,
                                   int32_t n_max, void* scratch, float* d_out, float* score, uint8_t* keep, cudaStream_t s);

}  // namespace dl
