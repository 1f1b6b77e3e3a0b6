// Host side of the C ABI: argument checks, workspace layout, dispatch to the kernel launchers.
// No call here allocates device memory or synchronises, except where dl.h says so.
#include <new>
#include <string.h>

#include "common.cuh"

namespace dl {

static inline int64_t align256(int64_t v) { return (v + 255) & ~int64_t(255); }

int64_t workspace_layout(const dl_model_desc& d, int32_t max_batch, int32_t max_rows, int32_t cap,
                         Workspace* ws) {
  int64_t off = 0;
  auto take = [&](int64_t bytes) { int64_t o = off; off = align256(off + bytes); return o; };
  const int64_t o_status = take(sizeof(DeviceStatus));
  const int64_t o_pbase = take((int64_t)max_batch * 4);
  const int64_t o_pcount = take((int64_t)max_batch * 4);
  const int64_t o_ticket = take((int64_t)kDecodeScratchSets * max_batch * d.n_heads * 4);
  const int32_t slots = (cap + kDecodeMinChunk - 1) / kDecodeMinChunk + 1;
  const int64_t o_partial = take((int64_t)kDecodeScratchSets * max_batch * d.n_heads * slots * (d.head_dim + 2) * 4);
  const int32_t rows_pad = (max_rows + kPredRowTile - 1) / kPredRowTile * kPredRowTile;
  const int64_t o_ppart = take((int64_t)kPredMaxSplit * rows_pad * 4);
  const int64_t o_ptick = take((int64_t)(rows_pad / kPredRowTile + 1) * 4);
  const int64_t o_psplit = take((int64_t)d.pred_hidden * kPredKSplit * kPredRowTile * 4);
  const int64_t o_pstick = take((int64_t)kPredMaxSplit * 4);
  const int64_t o_commit = take(2 * 4);
  const int64_t o_ones = take(max_batch);
  if (ws) {
    char* b = ws->base;
    ws->status = reinterpret_cast<DeviceStatus*>(b + o_status);
    ws->plan_base = reinterpret_cast<int32_t*>(b + o_pbase);
    ws->plan_count = reinterpret_cast<int32_t*>(b + o_pcount);
    ws->dec_ticket = reinterpret_cast<int32_t*>(b + o_ticket);
    ws->dec_partial = reinterpret_cast<float*>(b + o_partial);
    ws->dec_slots = slots;
    ws->pred_partial = reinterpret_cast<float*>(b + o_ppart);
    ws->pred_ticket = reinterpret_cast<int32_t*>(b + o_ptick);
    ws->pred_split = reinterpret_cast<float*>(b + o_psplit);
    ws->pred_split_ticket = reinterpret_cast<int32_t*>(b + o_pstick);
    ws->dec_commit = reinterpret_cast<int32_t*>(b + o_commit);
    ws->ones = reinterpret_cast<uint8_t*>(b + o_ones);
    ws->pred_rows_padded = rows_pad;
    ws->max_batch = max_batch; ws->max_rows = max_rows; ws->cap = cap;
  }
  return off;
}

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) { cudaSetDevice(dev); changed = true; }
  }
  ~DeviceGuard() { if (changed) cudaSetDevice(prev); }
};

static inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static inline int32_t cuda_status(dl_ctx* ctx, cudaError_t e) {
  if (e == cudaSuccess) return DL_OK;
  ctx->last_cuda = e;
  return DL_ERR_CUDA;
}

static inline int elt_bytes(const dl_ctx* ctx) { return ctx->desc.dtype == DL_F32 ? 4 : 2; }

// *keep_done (if given) tells whether the launch also wrote keep = score > threshold
static int32_t run_predictor(dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows, float* score,
                             cudaStream_t s, uint8_t* keep = nullptr, float threshold = 0.f, bool* keep_done = nullptr) {
  if (keep_done) *keep_done = false;
  if (!p || !p->w1 || !p->b1 || !p->w2 || !x || !score) return DL_ERR_INVALID_ARG;
  if (misaligned(p->w1) || misaligned(x)) return DL_ERR_ALIGNMENT;
  int impl = ctx->opt.predictor_impl;
  if (impl == 0) impl = predictor_tc_supported(ctx) ? 2 : 1;
  if (impl == 2) {
    if (!predictor_tc_supported(ctx)) return DL_ERR_UNSUPPORTED;
    if (!ctx->ws.base || rows > ctx->ws.max_rows) return DL_ERR_WORKSPACE;
    if (keep_done) *keep_done = keep != nullptr;
    return cuda_status(ctx, launch_predictor_tc(ctx, p, x, rows, score, s, keep, threshold));
  }
  return cuda_status(ctx, launch_predictor_simt(ctx, p, x, rows, score, s));
}

}  // namespace dl

using namespace dl;

extern "C" {

int32_t dl_create(dl_ctx** out, int32_t device, const dl_model_desc* desc) {
  if (!out || !desc) return DL_ERR_INVALID_ARG;
  *out = nullptr;
  if (desc->hidden <= 0 || desc->n_heads <= 0 || desc->pred_hidden <= 0) return DL_ERR_INVALID_ARG;
  if (desc->dtype != DL_F32 && desc->dtype != DL_BF16) return DL_ERR_UNSUPPORTED;
  if (desc->head_dim != 64 && desc->head_dim != 128) return DL_ERR_UNSUPPORTED;
  if (desc->hidden % 8 != 0) return DL_ERR_UNSUPPORTED;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return DL_ERR_CUDA;
  dl_ctx* c = new (std::nothrow) dl_ctx();
  if (!c) return DL_ERR_INVALID_ARG;
  c->device = device;
  c->desc = *desc;
  DeviceGuard g(device);
  int v = 0;
  cudaError_t e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) { c->sm_count = v; e = cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, device); }
  if (e != cudaSuccess) { delete c; return DL_ERR_CUDA; }
  c->smem_optin = v;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    c->tmap_encode = fn;
  (void)cudaGetLastError();
  *out = c;
  return DL_OK;
}

int32_t dl_destroy(dl_ctx* ctx) {
  if (ctx) {
    DeviceGuard g(ctx->device);
    if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
    if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
    for (int i = 0; i < 2; ++i) {
      if (ctx->ev_in[i]) cudaEventDestroy(ctx->ev_in[i]);
      if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
      if (ctx->ev_out[i]) cudaEventDestroy(ctx->ev_out[i]);
    }
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  }
  delete ctx;
  return DL_OK;
}

int64_t dl_workspace_bytes(const dl_ctx* ctx, int32_t max_batch, int32_t max_rows, int32_t cap) {
  if (!ctx || max_batch <= 0 || max_rows < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  return workspace_layout(ctx->desc, max_batch, max_rows, cap, nullptr);
}

int32_t dl_set_workspace(dl_ctx* ctx, void* dev_ptr, int64_t bytes, int32_t max_batch, int32_t max_rows,
                         int32_t cap, void* stream) {
  if (!ctx || !dev_ptr || max_batch <= 0 || max_rows < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev_ptr) & 255u) return DL_ERR_ALIGNMENT;
  const int64_t need = workspace_layout(ctx->desc, max_batch, max_rows, cap, nullptr);
  if (bytes < need) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  ctx->ws = Workspace();
  ctx->ws.base = static_cast<char*>(dev_ptr);
  ctx->ws.bytes = bytes;
  workspace_layout(ctx->desc, max_batch, max_rows, cap, &ctx->ws);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(ctx->ws.status, 0, sizeof(DeviceStatus), s);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ctx->ws.dec_ticket, 0, (size_t)kDecodeScratchSets * max_batch * ctx->desc.n_heads * 4, s);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ctx->ws.pred_ticket, 0, (size_t)(ctx->ws.pred_rows_padded / kPredRowTile + 1) * 4, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.dec_commit, 0, 2 * 4, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.pred_split_ticket, 0, (size_t)kPredMaxSplit * 4, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.ones, 1, (size_t)max_batch, s);
  return cuda_status(ctx, e);
}

int32_t dl_set_option(dl_ctx* ctx, int32_t option, int32_t value) {
  if (!ctx || value < 0) return DL_ERR_INVALID_ARG;
  switch (option) {
    case DL_OPT_PREDICTOR_IMPL: if (value > 2) return DL_ERR_INVALID_ARG; ctx->opt.predictor_impl = value; break;
    case DL_OPT_PREFILL_ATTN_IMPL: if (value > 2) return DL_ERR_INVALID_ARG; ctx->opt.prefill_attn_impl = value; break;
    case DL_OPT_DECODE_CHUNK: ctx->opt.decode_chunk = value; break;
    case DL_OPT_DECODE_IMPL: if (value > 2) return DL_ERR_INVALID_ARG; ctx->opt.decode_impl = value; break;
    case DL_OPT_COMPACT_IMPL: if (value > 2) return DL_ERR_INVALID_ARG; ctx->opt.compact_impl = value; break;
    default: return DL_ERR_INVALID_ARG;
  }
  return DL_OK;
}

int32_t dl_device_status(dl_ctx* ctx, void* stream, int32_t* code_out, int64_t* detail_out) {
  if (!ctx || !code_out) return DL_ERR_INVALID_ARG;
  if (!ctx->ws.base) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  DeviceStatus h;
  cudaError_t e = cudaMemcpyAsync(&h, ctx->ws.status, sizeof(h), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws.status, 0, sizeof(DeviceStatus), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(ctx, e);
  *code_out = h.code;
  if (detail_out) *detail_out = (int64_t)h.detail;
  return DL_OK;
}

const char* dl_status_str(int32_t status) {
  switch (status) {
    case DL_OK: return "ok";
    case DL_ERR_INVALID_ARG: return "invalid argument";
    case DL_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case DL_ERR_UNSUPPORTED: return "unsupported dtype, head_dim or size";
    case DL_ERR_WORKSPACE: return "workspace missing or too small";
    case DL_ERR_CUDA: return "CUDA runtime error";
    case DL_ERR_CAPACITY: return "kept rows do not fit into the cache";
    case DL_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case DL_ERR_BOUNDS: return "checked build: an index fell outside its buffer (access skipped)";
    case DL_WARN_NAN: return "NaN score ranked as -inf / dropped";
    default: return "unknown status";
  }
}

const char* dl_last_cuda_error(const dl_ctx* ctx) {
  return ctx ? cudaGetErrorString(ctx->last_cuda) : "no context";
}

int32_t dl_predictor_scores(dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows, float* score_out,
                            void* stream) {
  if (!ctx || rows < 0) return DL_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (rows == 0) return DL_OK;
  return run_predictor(ctx, p, x, rows, score_out, static_cast<cudaStream_t>(stream));
}

int32_t dl_topk_from_scores(dl_ctx* ctx, const float* score, const int32_t* n_vis, const int32_t* k, int32_t B,
                            int32_t n_vis_max, int32_t* kept_idx_out, int32_t k_max, uint8_t* keep_out,
                            void* stream) {
  if (!ctx || B < 0 || n_vis_max < 0 || k_max < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_vis_max == 0) return DL_OK;
  if (!score || !k || !keep_out) return DL_ERR_INVALID_ARG;
  if (n_vis_max > 16384) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_topk(score, n_vis, k, B, n_vis_max, kept_idx_out, k_max, keep_out,
                                      ctx->ws.status, static_cast<cudaStream_t>(stream)));
}

int32_t dl_prefill_select(dl_ctx* ctx, const dl_predictor* p_img, const void* x_vis, const int32_t* n_vis,
                          const int32_t* k, int32_t B, int32_t n_vis_max, float* score_out,
                          int32_t* kept_idx_out, int32_t k_max, uint8_t* keep_out, void* stream) {
  if (!ctx || B < 0 || n_vis_max < 0 || k_max < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_vis_max == 0) return DL_OK;
  if ((int64_t)B * n_vis_max > INT32_MAX) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  int32_t st = run_predictor(ctx, p_img, x_vis, B * n_vis_max, score_out, static_cast<cudaStream_t>(stream));
  if (st != DL_OK) return st;
  return dl_topk_from_scores(ctx, score_out, n_vis, k, B, n_vis_max, kept_idx_out, k_max, keep_out, stream);
}

int64_t dl_predictor2_scratch_bytes(const dl_ctx* ctx, int64_t rows) {
  if (!ctx || rows < 0) return DL_ERR_INVALID_ARG;
  return predictor_paper_scratch_bytes(rows);
}

static int32_t check_predictor2(const dl_ctx* ctx, const dl_predictor2* p) {
  if (!p || !p->in.w || !p->in.b || !p->h1.w || !p->h1.b || !p->h2.w || !p->h2.b || !p->w3 || !p->b3) return DL_ERR_INVALID_ARG;
  if (p->n_blocks < 0 || p->n_blocks > 16 || (p->n_blocks > 0 && !p->blocks)) return DL_ERR_INVALID_ARG;
  for (int i = 0; i < p->n_blocks; ++i) {
    const dl_vit_block& k = p->blocks[i];
    if (!k.ln1_g || !k.ln1_b || !k.ln2_g || !k.ln2_b || !k.qkv.w || !k.qkv.b || !k.proj.w || !k.proj.b || !k.fc1.w ||
        !k.fc1.b || !k.fc2.w || !k.fc2.b)
      return DL_ERR_INVALID_ARG;
    if (misaligned(k.qkv.w) || misaligned(k.proj.w) || misaligned(k.fc1.w) || misaligned(k.fc2.w) ||
        misaligned(k.ln1_g) || misaligned(k.ln1_b) || misaligned(k.ln2_g) || misaligned(k.ln2_b))
      return DL_ERR_ALIGNMENT;
  }
  if (misaligned(p->in.w) || misaligned(p->h1.w) || misaligned(p->h2.w) || misaligned(p->w3)) return DL_ERR_ALIGNMENT;
  return predictor_paper_supported(ctx) ? DL_OK : DL_ERR_UNSUPPORTED;
}

int32_t dl_predictor2_values(dl_ctx* ctx, const dl_predictor2* p, const void* x, const int32_t* n_vis, int32_t B, int32_t n_max,
                      void* scratch, int64_t scratch_bytes, float* d_out, float* score_out, uint8_t* keep_out, void* stream) {
  if (!ctx || B < 0 || n_max < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_max == 0) return DL_OK;
  if ((int64_t)B * n_max > INT32_MAX / 4) return DL_ERR_UNSUPPORTED;
  int32_t st = check_predictor2(ctx, p);
  if (st != DL_OK) return st;
  if (!x || !scratch) return DL_ERR_INVALID_ARG;
  if (misaligned(x) || (reinterpret_cast<uintptr_t>(scratch) & 255u)) return DL_ERR_ALIGNMENT;
  if (scratch_bytes < predictor_paper_scratch_bytes((int64_t)B * n_max)) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_predictor_paper(ctx, p, x, n_vis, B, n_max, scratch, d_out, score_out, keep_out,
                                                 static_cast<cudaStream_t>(stream)));
}

int32_t dl_prefill_select2(dl_ctx* ctx, const dl_predictor2* p_img, const void* x_vis, const int32_t* n_vis,
                           const int32_t* k, int32_t B, int32_t n_vis_max, void* scratch, int64_t scratch_bytes,
                           float* d_out, float* score_out, int32_t* kept_idx_out, int32_t k_max, uint8_t* keep_out,
                           void* stream) {
  if (!score_out) return DL_ERR_INVALID_ARG;
  int32_t st = dl_predictor2_values(ctx, p_img, x_vis, n_vis, B, n_vis_max, scratch, scratch_bytes, d_out, score_out, nullptr, stream);
  if (st != DL_OK) return st;
  return dl_topk_from_scores(ctx, score_out, n_vis, k, B, n_vis_max, kept_idx_out, k_max, keep_out, stream);
}

int32_t dl_decode_keep2(dl_ctx* ctx, const dl_predictor2* p_txt, const void* x_t, int32_t B, void* scratch,
                        int64_t scratch_bytes, float* d_out, uint8_t* keep_out, void* stream) {
  if (!keep_out || (p_txt && p_txt->n_blocks != 0)) return DL_ERR_INVALID_ARG;
  return dl_predictor2_values(ctx, p_txt, x_t, nullptr, B, 1, scratch, scratch_bytes, d_out, nullptr, keep_out, stream);
}

int32_t dl_compact_kv(dl_ctx* ctx, const void* k_src, const void* v_src, const uint8_t* keep,
                      int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache, void* v_cache,
                      int32_t cap, int32_t* cache_len, int32_t commit, void* stream) {
  if (!ctx || B < 0 || t_src_max < 0 || cap <= 0 || keep_cols < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || t_src_max == 0) return DL_OK;
  if (!k_src || !k_cache || !cache_len) return DL_ERR_INVALID_ARG;
  if ((v_src == nullptr) != (v_cache == nullptr)) return DL_ERR_INVALID_ARG;
  if (misaligned(k_src) || misaligned(v_src) || misaligned(k_cache) || misaligned(v_cache)) return DL_ERR_ALIGNMENT;
  if (!ctx->ws.base || B > ctx->ws.max_batch) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_compact(ctx, k_src, v_src, keep, keep_cols, t_src, B, t_src_max, k_cache, v_cache, cap,
                                         cache_len, commit, static_cast<cudaStream_t>(stream)));
}

int32_t dl_compact_kv_layers(dl_ctx* ctx, int32_t n_tensors, const void* const* srcs, void* const* caches,
                             const uint8_t* keep, int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max,
                             int32_t cap, int32_t* cache_len, int32_t commit, void* stream) {
  if (!ctx || n_tensors < 0 || B < 0 || t_src_max < 0 || cap <= 0 || keep_cols < 0) return DL_ERR_INVALID_ARG;
  if (n_tensors == 0 || B == 0 || t_src_max == 0) return DL_OK;
  if (!srcs || !caches || !cache_len) return DL_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n_tensors; ++i) {
    if (!srcs[i] || !caches[i]) return DL_ERR_INVALID_ARG;
    if (misaligned(srcs[i]) || misaligned(caches[i])) return DL_ERR_ALIGNMENT;
  }
  if (!ctx->ws.base || B > ctx->ws.max_batch) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // one plan, then the tensors two by two: every copy launch lets the next one start while it drains and
  // waits for its predecessor before it ends
  const int32_t launches = (n_tensors + 1) / 2;
  for (int32_t l = 0; l < launches; ++l) {
    const void* v_src = 2 * l + 1 < n_tensors ? srcs[2 * l + 1] : nullptr;
    void* v_cache = 2 * l + 1 < n_tensors ? caches[2 * l + 1] : nullptr;
    const int32_t chained = launches > 1 ? (1 | (l > 0 ? 2 : 0)) : 0;
    cudaError_t e = launch_compact(ctx, srcs[2 * l], v_src, keep, keep_cols, t_src, B, t_src_max, caches[2 * l], v_cache,
                                   cap, cache_len, commit, s, 0, l > 0, chained);
    if (e != cudaSuccess) return cuda_status(ctx, e);
  }
  return DL_OK;
}

// The device's address of a pinned, device-reachable host buffer (nullptr if it is anything else).
static const void* device_view_of_host(const void* host_ptr) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) return nullptr;
  return at.devicePointer;
}

int32_t dl_compact_kv_host(dl_ctx* ctx, const void* k_src_host, const void* v_src_host, const uint8_t* keep,
                           int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                           void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, void* stream) {
  if (!ctx || B < 0 || t_src_max < 0 || cap <= 0 || keep_cols < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || t_src_max == 0) return DL_OK;
  if (!k_src_host || !k_cache || !cache_len) return DL_ERR_INVALID_ARG;
  if ((v_src_host == nullptr) != (v_cache == nullptr)) return DL_ERR_INVALID_ARG;
  if (!ctx->ws.base || B > ctx->ws.max_batch) return DL_ERR_WORKSPACE;
  DeviceGuard g(ctx->device);
  const void* k_dev = device_view_of_host(k_src_host);
  const void* v_dev = v_src_host ? device_view_of_host(v_src_host) : nullptr;
  if (!k_dev || (v_src_host && !v_dev)) return DL_ERR_INVALID_ARG;      // not pinned host memory
  if (misaligned(k_dev) || misaligned(v_dev) || misaligned(k_cache) || misaligned(v_cache)) return DL_ERR_ALIGNMENT;
  // the copy kernel with plain 16-byte loads: they reach pinned host memory like any other address
  return cuda_status(ctx, launch_compact(ctx, k_dev, v_dev, keep, keep_cols, t_src, B, t_src_max, k_cache, v_cache, cap,
                                         cache_len, commit, static_cast<cudaStream_t>(stream), 1));
}

int32_t dl_sparse_attn_prefill(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max, float scale,
                               void* out, void* stream) {
  if (!ctx || B < 0 || cap <= 0 || n_max < 0 || n_max > cap || !(scale > 0.f)) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_max == 0) return DL_OK;
  if (!q || !k_cache || !v_cache || !cache_len || !out) return DL_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k_cache) || misaligned(v_cache) || misaligned(out)) return DL_ERR_ALIGNMENT;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int impl = ctx->opt.prefill_attn_impl;
  if (impl == 0) impl = attn_prefill_tc_supported(ctx) ? 2 : 1;
  if (impl >= 2) {
    if (!attn_prefill_tc_supported(ctx)) return DL_ERR_UNSUPPORTED;
    return cuda_status(ctx, launch_attn_prefill_tc(ctx, q, k_cache, v_cache, cache_len, B, cap, n_max, scale, out, s));
  }
  return cuda_status(ctx, launch_attn_prefill_simt(ctx, q, k_cache, v_cache, cache_len, B, cap, n_max, scale, out, s));
}

// One layer's decode attention.  `overlap_prev`: the launch may begin while the previous kernel of
// the stream is still draining (only dl_decode_step asks for it, for layers 1.. of a stack whose
// caches and outputs are distinct tensors).
static int32_t decode_layer(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t, void* k_cache,
                            void* v_cache, const int32_t* cache_len, const uint8_t* keep, int32_t B,
                            int32_t cap, float scale, void* out, bool overlap_prev, int scratch_set, void* stream,
                            int32_t* commit_len = nullptr, int commit_slot = 0) {
  if (!ctx || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!q_t || !k_t || !v_t || !k_cache || !v_cache || !cache_len || !out) return DL_ERR_INVALID_ARG;
  if (misaligned(q_t) || misaligned(k_t) || misaligned(v_t) || misaligned(k_cache) || misaligned(v_cache) ||
      misaligned(out))
    return DL_ERR_ALIGNMENT;
  if (!ctx->ws.base || B > ctx->ws.max_batch || cap > ctx->ws.cap) return DL_ERR_WORKSPACE;
  if (B > 2048) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_attn_decode(ctx, q_t, k_t, v_t, k_cache, v_cache, cache_len, keep, B, cap,
                                             scale, out, overlap_prev, scratch_set, static_cast<cudaStream_t>(stream),
                                             commit_len, commit_slot));
}

int32_t dl_sparse_attn_decode(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t, void* k_cache,
                              void* v_cache, const int32_t* cache_len, const uint8_t* keep, int32_t B,
                              int32_t cap, float scale, void* out, void* stream) {
  return decode_layer(ctx, q_t, k_t, v_t, k_cache, v_cache, cache_len, keep, B, cap, scale, out, false, 0, stream);
}

int32_t dl_quantize_kv_fp8(dl_ctx* ctx, const void* src, const int32_t* cache_len, const float* scale, int32_t B,
                           int32_t cap, void* dst, void* stream) {
  if (!ctx || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!src || !cache_len || !scale || !dst) return DL_ERR_INVALID_ARG;
  if (misaligned(src) || misaligned(dst)) return DL_ERR_ALIGNMENT;
  if (ctx->desc.dtype != DL_BF16 || ctx->desc.head_dim != 128) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_quantize_kv_fp8(ctx, src, cache_len, scale, B, cap, dst,
                                                 static_cast<cudaStream_t>(stream)));
}

int32_t dl_sparse_attn_decode_fp8(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t, void* k_cache,
                                  void* v_cache, const float* k_scale, const float* v_scale,
                                  const int32_t* cache_len, const uint8_t* keep, int32_t B, int32_t cap, float scale,
                                  void* out, void* stream) {
  if (!ctx || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!q_t || !k_t || !v_t || !k_cache || !v_cache || !k_scale || !v_scale || !cache_len || !out)
    return DL_ERR_INVALID_ARG;
  if (misaligned(q_t) || misaligned(k_t) || misaligned(v_t) || misaligned(k_cache) || misaligned(v_cache) ||
      misaligned(out))
    return DL_ERR_ALIGNMENT;
  if (ctx->desc.dtype != DL_BF16 || ctx->desc.head_dim != 128 || !ctx->tmap_encode) return DL_ERR_UNSUPPORTED;
  if (!ctx->ws.base || B > ctx->ws.max_batch || cap > ctx->ws.cap) return DL_ERR_WORKSPACE;
  if (B > 2048) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_attn_decode_fp8(ctx, q_t, k_t, v_t, k_cache, v_cache, k_scale, v_scale, cache_len,
                                                 keep, B, cap, scale, out, static_cast<cudaStream_t>(stream)));
}

int32_t dl_sparse_attn_decode_fp8_layers(dl_ctx* ctx, int32_t L, const void* q_t, const void* k_t, const void* v_t,
                                         void* const* k_caches, void* const* v_caches, const float* k_scales,
                                         const float* v_scales, int32_t* cache_len, const uint8_t* keep, int32_t B,
                                         int32_t cap, float scale, void* out, int32_t commit, void* stream) {
  if (!ctx || L < 0 || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || L == 0) return DL_OK;
  if (!q_t || !k_t || !v_t || !k_caches || !v_caches || !k_scales || !v_scales || !cache_len || !out)
    return DL_ERR_INVALID_ARG;
  if (commit && !keep) return DL_ERR_INVALID_ARG;
  const size_t layer_bytes = (size_t)B * ctx->desc.n_heads * ctx->desc.head_dim * elt_bytes(ctx);
  for (int32_t l = 0; l < L; ++l) {
    const char* ql = static_cast<const char*>(q_t) + l * layer_bytes;
    const char* kl = static_cast<const char*>(k_t) + l * layer_bytes;
    const char* vl = static_cast<const char*>(v_t) + l * layer_bytes;
    char* ol = static_cast<char*>(out) + l * layer_bytes;
    if (!k_caches[l] || !v_caches[l]) return DL_ERR_INVALID_ARG;
    if (misaligned(ql) || misaligned(k_caches[l]) || misaligned(v_caches[l]) || misaligned(ol)) return DL_ERR_ALIGNMENT;
    if (ctx->desc.dtype != DL_BF16 || ctx->desc.head_dim != 128 || !ctx->tmap_encode) return DL_ERR_UNSUPPORTED;
    if (!ctx->ws.base || B > ctx->ws.max_batch || cap > ctx->ws.cap) return DL_ERR_WORKSPACE;
    if (B > 2048) return DL_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    // consecutive layers touch different caches and outputs, so layer l may start while layer l-1 drains
    const bool overlap = l > 0 && k_caches[l] != k_caches[l - 1] && v_caches[l] != v_caches[l - 1];
    const int32_t st = cuda_status(ctx, launch_attn_decode_fp8(
        ctx, ql, kl, vl, k_caches[l], v_caches[l], k_scales + (size_t)l * ctx->desc.n_heads,
        v_scales + (size_t)l * ctx->desc.n_heads, cache_len, keep, B, cap, scale, ol,
        static_cast<cudaStream_t>(stream), L > 1, overlap, l % kDecodeScratchSets));
    if (st != DL_OK) return st;
  }
  // every layer has appended with the shared decision: the lengths advance once (stream order: after the last layer,
  // whose grid-dependency wait means all earlier layers are complete too)
  if (commit) return dl_commit_len(ctx, keep, B, cap, cache_len, stream);
  return DL_OK;
}

int32_t dl_decode_keep(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B, float threshold,
                       float* logit_inout, uint8_t* keep_out, void* stream) {
  if (!ctx || B < 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!logit_inout || !keep_out) return DL_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (x_t) {
    // the tensor-core predictor takes the decision where it completes the logit: no second launch
    bool keep_done = false;
    int32_t st = run_predictor(ctx, p_txt, x_t, B, logit_inout, s, keep_out, threshold, &keep_done);
    if (st != DL_OK || keep_done) return st;
  }
  return cuda_status(ctx, launch_decode_keep(logit_inout, B, threshold, keep_out, ctx->ws.status, s));
}

int32_t dl_decode_nocache_select(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_gen, const int32_t* n_gen,
                                 int32_t B, int32_t n_gen_max, float threshold, float* logit_inout,
                                 uint8_t* keep_out, void* stream) {
  if (!ctx || B < 0 || n_gen_max < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_gen_max == 0) return DL_OK;
  if (!logit_inout || !keep_out) return DL_ERR_INVALID_ARG;
  if ((int64_t)B * n_gen_max > INT32_MAX) return DL_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (x_gen) {
    int32_t st = run_predictor(ctx, p_txt, x_gen, B * n_gen_max, logit_inout, s);
    if (st != DL_OK) return st;
  }
  return cuda_status(ctx, launch_nocache_mask(logit_inout, n_gen, B, n_gen_max, threshold, keep_out,
                                              ctx->ws.status, s));
}

int32_t dl_commit_len(dl_ctx* ctx, const uint8_t* keep, int32_t B, int32_t cap, int32_t* cache_len,
                      void* stream) {
  if (!ctx || B < 0 || cap <= 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!keep || !cache_len) return DL_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  return cuda_status(ctx, launch_commit_len(keep, B, cap, cache_len, static_cast<cudaStream_t>(stream)));
}

// Layers [l0, l1) of a decode step's stack, all with the same lengths, decision and capacity.  q_t, k_t, v_t, out
// and the cache arrays are those of the whole stack (indexed by layer).  commit_len (null or the lengths, writable):
// the launch of layer l1 - 1 also closes the step for these layers, cache_len[b] += keep[b], once every launch of the
// group has read the lengths for the last time; groups in flight together use different commit slots.
static int32_t decode_layer_range(dl_ctx* ctx, int32_t l0, int32_t l1, const void* q_t, const void* k_t,
                                  const void* v_t, void* const* k_caches, void* const* v_caches,
                                  const int32_t* cache_len, const uint8_t* keep, int32_t B, int32_t cap, float scale,
                                  void* out, void* stream, int32_t* commit_len, int commit_slot) {
  const size_t layer_bytes = (size_t)B * ctx->desc.n_heads * ctx->desc.head_dim * elt_bytes(ctx);
  for (int32_t l = l0; l < l1; ++l) {
    const char* ql = static_cast<const char*>(q_t) + l * layer_bytes;
    const char* kl = static_cast<const char*>(k_t) + l * layer_bytes;
    const char* vl = static_cast<const char*>(v_t) + l * layer_bytes;
    char* ol = static_cast<char*>(out) + l * layer_bytes;
    // consecutive layers touch different caches and outputs, so layer l may start while layer l-1 drains
    const bool overlap = l > 0 && k_caches[l] != k_caches[l - 1] && v_caches[l] != v_caches[l - 1];
    int32_t st = decode_layer(ctx, ql, kl, vl, k_caches[l], v_caches[l], cache_len, keep, B, cap, scale, ol, overlap,
                              l % kDecodeScratchSets, stream, l == l1 - 1 ? commit_len : nullptr, commit_slot);
    if (st != DL_OK) return st;
  }
  return DL_OK;
}

static int32_t decode_layers(dl_ctx* ctx, int32_t L, const void* q_t, const void* k_t, const void* v_t,
                             void* const* k_caches, void* const* v_caches, const int32_t* cache_len,
                             const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out, void* stream,
                             int32_t* commit_len) {
  if (!ctx || L < 0 || B < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || L == 0) return DL_OK;
  if (!k_caches || !v_caches || !q_t || !k_t || !v_t || !out) return DL_ERR_INVALID_ARG;
  ctx->opt.in_layer_stack = L > 1 ? 1 : 0;
  const int32_t st = decode_layer_range(ctx, 0, L, q_t, k_t, v_t, k_caches, v_caches, cache_len, keep, B, cap, scale,
                                        out, stream, commit_len, 0);
  ctx->opt.in_layer_stack = 0;
  return st;
}

int32_t dl_sparse_attn_decode_layers(dl_ctx* ctx, int32_t L, const void* q_t, const void* k_t, const void* v_t,
                                     void* const* k_caches, void* const* v_caches, const int32_t* cache_len,
                                     const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                                     void* stream) {
  return decode_layers(ctx, L, q_t, k_t, v_t, k_caches, v_caches, cache_len, keep, B, cap, scale, out, stream, nullptr);
}

int32_t dl_decode_step(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B, float threshold,
                       float* logit_inout, uint8_t* keep_out, int32_t L, const void* q_t, const void* k_t,
                       const void* v_t, void* const* k_caches, void* const* v_caches, int32_t cap,
                       int32_t* cache_len, float scale, void* out, void* stream) {
  if (!ctx || L < 0 || B < 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (L > 0 && (!k_caches || !v_caches || !q_t || !k_t || !v_t || !out)) return DL_ERR_INVALID_ARG;
  int32_t st = dl_decode_keep(ctx, p_txt, x_t, B, threshold, logit_inout, keep_out, stream);
  if (st != DL_OK) return st;
  // the step is closed by its last attention launch; without layers the commit is a launch of its own
  if (L == 0) return dl_commit_len(ctx, keep_out, B, cap, cache_len, stream);
  if (!cache_len) return DL_ERR_INVALID_ARG;
  return decode_layers(ctx, L, q_t, k_t, v_t, k_caches, v_caches, cache_len, keep_out, B, cap, scale, out, stream,
                       cache_len);
}

int32_t dl_decode_step_stack(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B, float threshold,
                             float* logit_inout, uint8_t* keep_out, const dl_layer_stack* stack, const void* q_t,
                             const void* k_t, const void* v_t, float scale, void* out, void* stream) {
  if (!ctx || !stack || B < 0) return DL_ERR_INVALID_ARG;
  const int32_t L = stack->L, ld = stack->l_dense;
  if (L < 0 || ld < 0 || ld > L) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (L > 0 && (!stack->k_caches || !stack->v_caches || !q_t || !k_t || !v_t || !out)) return DL_ERR_INVALID_ARG;
  if ((ld > 0 && (!stack->len_dense || stack->cap_dense <= 0)) || (ld < L && (!stack->cache_len || stack->cap <= 0)))
    return DL_ERR_INVALID_ARG;
  if (!ctx->ws.base || B > ctx->ws.max_batch) return DL_ERR_WORKSPACE;
  int32_t st = dl_decode_keep(ctx, p_txt, x_t, B, threshold, logit_inout, keep_out, stream);
  if (st != DL_OK) return st;
  if (L == 0) return DL_OK;
  ctx->opt.in_layer_stack = L > 1 ? 1 : 0;
  // the dense layers keep every token: their decision is a vector of ones, their lengths grow by one per step
  if (ld > 0)
    st = decode_layer_range(ctx, 0, ld, q_t, k_t, v_t, stack->k_caches, stack->v_caches, stack->len_dense,
                            ctx->ws.ones, B, stack->cap_dense, scale, out, stream, stack->len_dense, 1);
  if (st == DL_OK && ld < L)
    st = decode_layer_range(ctx, ld, L, q_t, k_t, v_t, stack->k_caches, stack->v_caches, stack->cache_len, keep_out,
                            B, stack->cap, scale, out, stream, stack->cache_len, 0);
  ctx->opt.in_layer_stack = 0;
  return st;
}

int32_t dl_decode_step_host(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_host, int32_t B,
                            float threshold, int32_t L, const void* q_host, const void* k_host,
                            const void* v_host, void* out_host, uint8_t* keep_host, void* stage_x,
                            void* stage_q, void* stage_k, void* stage_v, void* stage_out, float* logit_dev,
                            uint8_t* keep_dev, void* const* k_caches, void* const* v_caches, int32_t cap,
                            int32_t* cache_len, float scale, void* stream) {
  if (!ctx || L < 0 || B < 0) return DL_ERR_INVALID_ARG;
  if (B == 0) return DL_OK;
  if (!x_host || !stage_x || !logit_dev || !keep_dev) return DL_ERR_INVALID_ARG;
  if (L > 0 && (!q_host || !k_host || !v_host || !out_host || !stage_q || !stage_k || !stage_v || !stage_out))
    return DL_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t xb = (size_t)B * ctx->desc.hidden * elt_bytes(ctx);
  const size_t lb = (size_t)L * B * ctx->desc.n_heads * ctx->desc.head_dim * elt_bytes(ctx);
  cudaError_t e = cudaMemcpyAsync(stage_x, x_host, xb, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && lb) e = cudaMemcpyAsync(stage_q, q_host, lb, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && lb) e = cudaMemcpyAsync(stage_k, k_host, lb, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && lb) e = cudaMemcpyAsync(stage_v, v_host, lb, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_status(ctx, e);
  int32_t st = dl_decode_step(ctx, p_txt, stage_x, B, threshold, logit_dev, keep_dev, L, stage_q, stage_k,
                              stage_v, k_caches, v_caches, cap, cache_len, scale, stage_out, stream);
  if (st != DL_OK) return st;
  if (lb) e = cudaMemcpyAsync(out_host, stage_out, lb, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess && keep_host) e = cudaMemcpyAsync(keep_host, keep_dev, (size_t)B, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return cuda_status(ctx, e);
}

// Copy streams and events of the pipelined host-fed decode: made once per context.
static cudaError_t host_pipeline_setup(dl_ctx* ctx) {
  if (ctx->h2d_stream) return cudaSuccess;
  cudaError_t e = cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
  return e;
}

int32_t dl_decode_steps_host(dl_ctx* ctx, const dl_predictor* p_txt, int32_t n_steps, int32_t B, float threshold,
                             int32_t L, const void* const* x_host, const void* const* q_host,
                             const void* const* k_host, const void* const* v_host, void* const* out_host,
                             uint8_t* const* keep_host, void* stage_x, void* stage_q, void* stage_k, void* stage_v,
                             void* stage_out, float* logit_dev, uint8_t* keep_dev, void* const* k_caches,
                             void* const* v_caches, int32_t cap, int32_t* cache_len, float scale, void* stream) {
  if (!ctx || n_steps < 0 || L < 0 || B < 0) return DL_ERR_INVALID_ARG;
  if (B == 0 || n_steps == 0) return DL_OK;
  if (!x_host || !stage_x || !logit_dev || !keep_dev) return DL_ERR_INVALID_ARG;
  if (L > 0 && (!q_host || !k_host || !v_host || !out_host || !stage_q || !stage_k || !stage_v || !stage_out))
    return DL_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = host_pipeline_setup(ctx);
  if (e != cudaSuccess) return cuda_status(ctx, e);
  cudaStream_t s = static_cast<cudaStream_t>(stream), sin = ctx->h2d_stream, sout = ctx->d2h_stream;
  const size_t xb = (size_t)B * ctx->desc.hidden * elt_bytes(ctx);
  const size_t lb = (size_t)L * B * ctx->desc.n_heads * ctx->desc.head_dim * elt_bytes(ctx);
  // the copy streams start behind whatever the caller has queued on `stream`
  e = cudaEventRecord(ctx->ev_fork, s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(sin, ctx->ev_fork, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(sout, ctx->ev_fork, 0);
  int32_t st = DL_OK;
  for (int32_t t = 0; t < n_steps && e == cudaSuccess && st == DL_OK; ++t) {
    const int set = t & 1;
    char* sx = static_cast<char*>(stage_x) + set * xb;
    char* sq = static_cast<char*>(stage_q) + set * lb;
    char* sk = static_cast<char*>(stage_k) + set * lb;
    char* sv = static_cast<char*>(stage_v) + set * lb;
    char* so = static_cast<char*>(stage_out) + set * lb;
    // inputs of step t into staging set `set`, once step t-2 has finished computing from it
    if (t >= 2) e = cudaStreamWaitEvent(sin, ctx->ev_done[set], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sx, x_host[t], xb, cudaMemcpyHostToDevice, sin);
    if (e == cudaSuccess && lb) e = cudaMemcpyAsync(sq, q_host[t], lb, cudaMemcpyHostToDevice, sin);
    if (e == cudaSuccess && lb) e = cudaMemcpyAsync(sk, k_host[t], lb, cudaMemcpyHostToDevice, sin);
    if (e == cudaSuccess && lb) e = cudaMemcpyAsync(sv, v_host[t], lb, cudaMemcpyHostToDevice, sin);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_in[set], sin);
    // the step itself, once its inputs have landed and step t-2's results have left the output staging
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->ev_in[set], 0);
    if (e == cudaSuccess && t >= 2) e = cudaStreamWaitEvent(s, ctx->ev_out[set], 0);
    if (e != cudaSuccess) break;
    st = dl_decode_step(ctx, p_txt, sx, B, threshold, logit_dev + (size_t)set * B, keep_dev + (size_t)set * B, L, sq,
                        sk, sv, k_caches, v_caches, cap, cache_len, scale, so, stream);
    if (st != DL_OK) break;
    e = cudaEventRecord(ctx->ev_done[set], s);
    // results of step t back to the host
    if (e == cudaSuccess) e = cudaStreamWaitEvent(sout, ctx->ev_done[set], 0);
    if (e == cudaSuccess && lb) e = cudaMemcpyAsync(out_host[t], so, lb, cudaMemcpyDeviceToHost, sout);
    if (e == cudaSuccess && keep_host && keep_host[t])
      e = cudaMemcpyAsync(keep_host[t], keep_dev + (size_t)set * B, (size_t)B, cudaMemcpyDeviceToHost, sout);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_out[set], sout);
  }
  // everything that was queued is waited for, also after an error (the staging buffers are the caller's)
  cudaError_t e1 = cudaStreamSynchronize(sin), e2 = cudaStreamSynchronize(s), e3 = cudaStreamSynchronize(sout);
  if (st != DL_OK) return st;
  if (e == cudaSuccess) e = e1 != cudaSuccess ? e1 : (e2 != cudaSuccess ? e2 : e3);
  return cuda_status(ctx, e);
}

}  // extern "C"
