/*
 * dl.h -- C ABI of the Dynamic-LLaVA sparsified-inference hot path for NVIDIA B200 (sm_100a).
 *
 * The calls follow the method's statement in the paper (arXiv 2412.00876):
 *   prefill  (Eq. 5, Eq. 11): a predictor scores every vision token, the k best are kept,
 *            the kept rows plus all text rows form the reduced set S^{P*}, and every later
 *            layer attends over that reduced set only (Eq. 1 on S^{P*});
 *   decoding with KV cache (Eq. 6): the current token always takes part in its own attention,
 *            and its K/V are appended to the cache only if the predictor's decision is 1;
 *            the decision is taken once per token and shared by all later layers (Sec. 3.3.1).
 *
 * Conventions
 *   - Plain C.  Every call returns an int32_t status: DL_OK (0) or a negative DL_ERR_*.
 *   - "dev" pointers are device memory owned by the caller; "host" pointers are host memory.
 *     The library allocates no device memory: scratch comes from the caller (dl_set_workspace).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     unless stated otherwise.  One context serves one stream at a time.
 *   - Tensors are dense, innermost dimension contiguous, every tensor pointer 16-byte aligned.
 *     Element type `dtype` (DL_F32 or DL_BF16) applies to activations, Q/K/V, caches, outputs
 *     and W1; scores, logits, b1, w2 are always float32.
 *   - Cache layout (what compaction is judged on, bit for bit): per layer, K and V are separate
 *     tensors [B][H][cap][D], D contiguous.  Rows [0, cache_len[b]) of sequence b are valid;
 *     rows beyond are unspecified.
 *   - Errors found on the device (capacity overflow, NaN score) are recorded in a status word
 *     inside the workspace; dl_device_status reads it back.  Nothing traps.
 */
#ifndef DL_SPARSE_H_
#define DL_SPARSE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dl_ctx dl_ctx;

enum { DL_F32 = 0, DL_BF16 = 1 };

enum {
  DL_OK = 0,
  DL_ERR_INVALID_ARG = -1,   /* NULL pointer, negative size, k out of range, ... */
  DL_ERR_ALIGNMENT = -2,     /* a tensor pointer is not 16-byte aligned */
  DL_ERR_UNSUPPORTED = -3,   /* dtype / head_dim / size combination not built */
  DL_ERR_WORKSPACE = -4,     /* workspace missing or too small for this call */
  DL_ERR_CUDA = -5,          /* a CUDA runtime call failed (see dl_last_cuda_error) */
  DL_ERR_CAPACITY = -6,      /* device status: kept rows did not fit into the cache */
  DL_ERR_TIMEOUT = -7,       /* device status: a bounded wait ran out */
  DL_ERR_BOUNDS = -8,        /* device status (checked build only): an index fell outside its buffer; the access was skipped */
  DL_WARN_NAN = 1            /* device status: a NaN score was ranked as -inf / dropped */
};

/* Implementation selectors for dl_set_option. */
enum {
  DL_OPT_PREDICTOR_IMPL = 1,    /* 0 auto, 1 CUDA-core kernel, 2 tcgen05 tensor-core kernel (bf16) */
  DL_OPT_PREFILL_ATTN_IMPL = 2, /* 0 auto, 1 CUDA-core kernel, 2 tcgen05 tensor-core kernel (bf16, D=128) */
  DL_OPT_DECODE_CHUNK = 3,      /* cache rows per decode work item (0 = chosen by the library) */
  DL_OPT_DECODE_IMPL = 4,       /* 0 auto, 1 CUDA-core kernel, 2 tensor-core (mma.sync) kernel (bf16, D=128) */
  DL_OPT_COMPACT_IMPL = 5       /* 0 auto, 1 register-staged copy kernel, 2 bulk-copy (TMA) kernel over even ranges of kept
                                 * rows with one tensor store per row (auto: 2 for up to 2048 sequences, else 1) */
};

typedef struct {
  int32_t hidden;      /* d: width of the hidden rows fed to the predictors */
  int32_t n_heads;     /* H (multi-head attention: as many K/V heads as query heads) */
  int32_t head_dim;    /* D: 64 or 128 */
  int32_t pred_hidden; /* width of the predictor's hidden layer */
  int32_t dtype;       /* DL_F32 or DL_BF16 */
} dl_model_desc;

/* One token predictor in per-token MLP form: score = w2 . GELU(W1 x + b1) + b2, GELU in its
 * exact erf form.  With a single output the score is at once the ranking value of Eq. 11 and
 * the folded two-way decision of Eq. 5 (keep iff score > 0). */
typedef struct {
  const void* w1;   /* dev [pred_hidden][hidden], dtype */
  const float* b1;  /* dev [pred_hidden] */
  const float* w2;  /* dev [pred_hidden] */
  float b2;
} dl_predictor;

/* ---- context ------------------------------------------------------------------------- */

/* Creates a context for `device` and `desc` (copied).  Host call; may initialise the CUDA
 * context.  DL_ERR_UNSUPPORTED for head_dim not in {64,128}, hidden % 8 != 0 or unknown dtype. */
int32_t dl_create(dl_ctx** out, int32_t device, const dl_model_desc* desc);
int32_t dl_destroy(dl_ctx* ctx);

/* Bytes of scratch the calls below need for up to `max_batch` sequences, `max_rows` predictor
 * rows per call (B * n_vis_max in prefill) and caches of `cap` rows.  Negative on bad args. */
int64_t dl_workspace_bytes(const dl_ctx* ctx, int32_t max_batch, int32_t max_rows, int32_t cap);

/* Hands the context its scratch (dev, 256-byte aligned, caller keeps ownership) and clears the
 * part that must start at zero (asynchronously on `stream`).  The sizes are the ones that were
 * given to dl_workspace_bytes. */
int32_t dl_set_workspace(dl_ctx* ctx, void* dev_ptr, int64_t bytes, int32_t max_batch,
                         int32_t max_rows, int32_t cap, void* stream);

int32_t dl_set_option(dl_ctx* ctx, int32_t option, int32_t value);

/* Synchronises `stream`, copies the device status word back and clears it.  code_out gets
 * DL_OK, DL_ERR_CAPACITY, DL_ERR_TIMEOUT or DL_WARN_NAN; detail_out the sequence index or row. */
int32_t dl_device_status(dl_ctx* ctx, void* stream, int32_t* code_out, int64_t* detail_out);

const char* dl_status_str(int32_t status);
/* Text of the last CUDA error seen by this context (host string owned by the library). */
const char* dl_last_cuda_error(const dl_ctx* ctx);

/* ---- prefill: Eq. 5 / Eq. 11 --------------------------------------------------------- */

/* Predictor alone (first line of Eq. 5 / Eq. 11): score_out[r] for `rows` hidden rows.
 * x dev [rows][hidden] dtype; score_out dev [rows] float32. */
int32_t dl_predictor_scores(dl_ctx* ctx, const dl_predictor* p, const void* x, int32_t rows,
                            float* score_out, void* stream);

/* TopkArgmax_k of Eq. 11 on given scores.  For each sequence b the k[b] largest of its first
 * n_vis[b] scores are kept; between equal scores the lower index wins; -0 equals +0; NaN ranks
 * as -inf (and sets DL_WARN_NAN).
 *   score dev [B][n_vis_max]; n_vis dev [B] or NULL (= n_vis_max); k dev [B], 0 <= k[b] <= n_vis[b]
 *   (a larger k[b] is clamped to n_vis[b]); kept_idx_out dev [B][k_max] ascending, unused slots -1
 *   (may be NULL); keep_out dev [B][n_vis_max] 0/1 (padding slots 0).  n_vis_max <= 16384.
 *   k_max must cover every k[b]: where it does not, the index list holds the first k_max kept indices only
 *   (the mask is complete) and DL_ERR_INVALID_ARG is recorded in the status word with the sequence index. */
int32_t dl_topk_from_scores(dl_ctx* ctx, const float* score, const int32_t* n_vis, const int32_t* k,
                            int32_t B, int32_t n_vis_max, int32_t* kept_idx_out, int32_t k_max,
                            uint8_t* keep_out, void* stream);

/* Eq. 11 end to end: scores of all vision rows, then the selection above.
 *   x_vis dev [B][n_vis_max][hidden]; score_out dev [B][n_vis_max]; others as above. */
int32_t dl_prefill_select(dl_ctx* ctx, const dl_predictor* p_img, const void* x_vis,
                          const int32_t* n_vis, const int32_t* k, int32_t B, int32_t n_vis_max,
                          float* score_out, int32_t* kept_idx_out, int32_t k_max, uint8_t* keep_out,
                          void* stream);

/* ---- compaction: set builder of Eq. 5, reduced set of Eq. 11, append of Eq. 6 --------- */

/* Appends to each sequence's cache, in token order, the source rows whose keep flag is 1,
 * starting at row cache_len[b]; if `commit` != 0, cache_len[b] += number appended.
 *   k_src, v_src dev [B][t_src_max][H][D] (v_src and v_cache may both be NULL: one tensor only);
 *   keep dev [B][keep_cols] or NULL (= keep all): the flags of the first keep_cols source rows;
 *   source rows t >= keep_cols are always kept.  In prefill keep_cols is the number of vision
 *   slots, so that the mask is M^I followed by ones for the text rows (S^{I*} u S^T of Eq. 11);
 *   t_src dev [B] valid source rows or NULL (= t_src_max);
 *   k_cache, v_cache dev [B][H][cap][D]; cache_len dev [B], read, and written when commit != 0.
 * Rows are copied bit for bit.  A sequence whose kept rows do not fit (cache_len + count > cap)
 * is left untouched, its length unchanged, and DL_ERR_CAPACITY is recorded with its index.
 * Several layers that share one decision pass commit = 0 for all but the last layer's call.
 * Needs the workspace. */
int32_t dl_compact_kv(dl_ctx* ctx, const void* k_src, const void* v_src, const uint8_t* keep,
                      int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                      void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, void* stream);

/* The same for n_tensors tensors that share ONE decision (Sec. 3.3.1: the mask is made once and used by every
 * later layer): K, V (and Q or hidden rows) of all layers in one call.  One plan (count, capacity check, length
 * commit) and a run of copy launches that overlap one another's start-up and tail; everything queued after the
 * call still finds all copies complete.  Same result, bit for bit, as n_tensors single-tensor calls of
 * dl_compact_kv with commit = 0 followed by the length commit.
 *   srcs, caches HOST arrays of n_tensors device pointers: srcs[i] [B][t_src_max][H][D] -> caches[i] [B][H][cap][D],
 *   every tensor appended at row cache_len[b]; the other arguments as for dl_compact_kv.  Needs the workspace. */
int32_t dl_compact_kv_layers(dl_ctx* ctx, int32_t n_tensors, const void* const* srcs, void* const* caches,
                             const uint8_t* keep, int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max,
                             int32_t cap, int32_t* cache_len, int32_t commit, void* stream);

/* dl_compact_kv with the SOURCE rows in pinned host memory (Eq. 5 / Eq. 11: only the kept rows enter the
 * reduced set, so only they need to reach the GPU).  The copy kernel reads the kept rows straight from host
 * memory over the bus; dropped rows never cross it, and no staging copy of the whole source is made.
 *   k_src_host, v_src_host HOST, pinned and reachable from the device (cudaHostAlloc / cudaHostRegister,
 *   e.g. torch's pin_memory()), [B][t_src_max][H][D]; every other argument as for dl_compact_kv (device).
 * The host buffers must stay valid and unchanged until the stream has passed this call.
 * DL_ERR_INVALID_ARG if a source is not such host memory. */
int32_t dl_compact_kv_host(dl_ctx* ctx, const void* k_src_host, const void* v_src_host, const uint8_t* keep,
                           int32_t keep_cols, const int32_t* t_src, int32_t B, int32_t t_src_max, void* k_cache,
                           void* v_cache, int32_t cap, int32_t* cache_len, int32_t commit, void* stream);

/* ---- attention over the reduced set --------------------------------------------------- */

/* Prefill (Eq. 1 on S^{P*}): causal scaled-dot-product attention of the compact rows against
 * themselves, per sequence and head: row i attends rows 0..i of the same cache.
 *   q dev [B][H][cap][D] compact queries in the cache layout (built by dl_compact_kv);
 *   k_cache, v_cache dev [B][H][cap][D]; cache_len dev [B]; n_max >= every cache_len[b], <= cap;
 *   out dev [B][n_max][H][D] (rows >= cache_len[b] are not written); scale > 0, usually 1/sqrt(D). */
int32_t dl_sparse_attn_prefill(dl_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* cache_len, int32_t B, int32_t cap, int32_t n_max,
                               float scale, void* out, void* stream);

/* Decoding with KV cache (Eq. 6, second line): Attention(Q, S^K u K, S^V u V) for one new token
 * per sequence: the query attends cache rows [0, cache_len[b]) plus the token's own (k_t, v_t).
 *   q_t, k_t, v_t dev [B][H][D]; out dev [B][H][D].
 * If `keep` (dev [B], may be NULL) is given, the call also performs Eq. 6's conditional append
 * for this layer: where keep[b] != 0, (k_t, v_t) are written to row cache_len[b] of the caches
 * (cache_len itself is not changed: call dl_commit_len once after the last layer).  A full
 * cache (cache_len[b] == cap) records DL_ERR_CAPACITY and skips the write.  Needs the workspace. */
int32_t dl_sparse_attn_decode(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t,
                              void* k_cache, void* v_cache, const int32_t* cache_len,
                              const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                              void* stream);

/* The same for a stack of L layers that share cache_len and keep (Eq. 6 applied per layer with the
 * one decision of Sec. 3.3.1): q_t, k_t, v_t, out dev [L][B][H][D]; k_caches, v_caches HOST arrays of
 * L device pointers, each [B][H][cap][D] and all distinct.  Equivalent to L calls of
 * dl_sparse_attn_decode in layer order, except that a layer's kernel may begin while the previous
 * layer's is still draining (they touch different caches and outputs); everything launched after
 * this call still sees all L layers complete. */
int32_t dl_sparse_attn_decode_layers(dl_ctx* ctx, int32_t L, const void* q_t, const void* k_t, const void* v_t,
                                     void* const* k_caches, void* const* v_caches, const int32_t* cache_len,
                                     const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                                     void* stream);

/* ---- decode decision: Eq. 5 applied to the current token (Eq. 6) ----------------------- */

/* logit[b] = P^{OT}(x_t[b]);  keep[b] = logit[b] > threshold (strict; NaN -> 0).
 *   x_t dev [B][hidden] or NULL: with NULL the logits already in logit_inout are used as given.
 *   logit_inout dev [B]; keep_out dev [B]. */
int32_t dl_decode_keep(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B,
                       float threshold, float* logit_inout, uint8_t* keep_out, void* stream);

/* Decoding WITHOUT KV cache (Eq. 12 and the sentence above Eq. 6): the decisions for ALL generated
 * tokens of every sequence at once; the last generated token of a sequence is always kept, since it
 * produces the next token.  keep[b][i] = i < n_gen[b] and (logit[b][i] > threshold or i == n_gen[b]-1).
 *   x_gen dev [B][n_gen_max][hidden] or NULL (then logit_inout is used as given); n_gen dev [B] or NULL
 *   (= n_gen_max); logit_inout dev [B][n_gen_max] float32; keep_out dev [B][n_gen_max] (padding 0).
 * The reduced set S^{P*} u S^{OT*} is then built with dl_compact_kv (this mask, keep_cols = n_gen_max,
 * t_src = n_gen, appended behind the compact prefill rows) and attended with dl_sparse_attn_prefill. */
int32_t dl_decode_nocache_select(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_gen, const int32_t* n_gen,
                                 int32_t B, int32_t n_gen_max, float threshold, float* logit_inout,
                                 uint8_t* keep_out, void* stream);

/* cache_len[b] += (keep[b] != 0) where cache_len[b] < cap: closes a decode step after every
 * layer has appended with the shared decision (Sec. 3.3.2). */
int32_t dl_commit_len(dl_ctx* ctx, const uint8_t* keep, int32_t B, int32_t cap, int32_t* cache_len,
                      void* stream);

/* One whole decode step over a stack of L layers that share the decision: dl_decode_keep, then
 * per layer dl_sparse_attn_decode with the fused append, then dl_commit_len.  Same results as those calls; the
 * library folds the decision into the predictor's launch and the length commit into the last layer's (1 + L
 * launches per step for bf16 models).
 *   q_t, k_t, v_t, out: dev [L][B][H][D]; k_caches, v_caches: HOST arrays of L device pointers,
 *   each [B][H][cap][D].  Other arguments as in the single calls. */
int32_t dl_decode_step(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B,
                       float threshold, float* logit_inout, uint8_t* keep_out, int32_t L,
                       const void* q_t, const void* k_t, const void* v_t, void* const* k_caches,
                       void* const* v_caches, int32_t cap, int32_t* cache_len, float scale,
                       void* out, void* stream);

/* A decoder's layer stack with the decision taken after its l-th layer (Sec. 3.3.1): the first l_dense layers run
 * before the decision exists and keep every token, the remaining L - l_dense share the decision.
 *   k_caches, v_caches: HOST arrays of L dev pointers; entries below l_dense are [B][H][cap_dense][D] caches whose
 *   lengths are len_dense (dev [B], +1 per step while below cap_dense), the others [B][H][cap][D] caches whose
 *   lengths are cache_len (dev [B], += keep per step).  The workspace must cover max(cap_dense, cap).
 *   len_dense may be NULL when l_dense == 0, cache_len when l_dense == L. */
typedef struct {
  int32_t L, l_dense;
  void* const* k_caches; void* const* v_caches;
  int32_t cap_dense, cap;
  int32_t* len_dense; int32_t* cache_len;
} dl_layer_stack;

/* dl_decode_step over such a stack (Eq. 6 with the layer placement of Sec. 3.3.1; with l_dense = 2 and one count of
 * image tokens this is the layer split Eq. 13's totals in Tab. 1 are made of): the decision, then one attention
 * launch per layer, dense layers first; the last dense launch advances len_dense, the last launch cache_len.
 *   q_t, k_t, v_t, out dev [L][B][H][D]. */
int32_t dl_decode_step_stack(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_t, int32_t B, float threshold,
                             float* logit_inout, uint8_t* keep_out, const dl_layer_stack* stack, const void* q_t,
                             const void* k_t, const void* v_t, float scale, void* out, void* stream);

/* The same step fed from HOST buffers (pinned for full copy speed): copies x_t, q_t, k_t, v_t
 * into the caller's device staging buffers, runs dl_decode_step, copies `out` and `keep` back to
 * the host, all on `stream`; returns after the stream has been synchronised.
 *   *_host: host counterparts of the dl_decode_step tensors; stage_* : dev buffers of the same
 *   sizes (x [B][hidden]; q, k, v, out [L][B][H][D]); logit_dev [B], keep_dev [B] dev. */
int32_t dl_decode_step_host(dl_ctx* ctx, const dl_predictor* p_txt, const void* x_host, int32_t B,
                            float threshold, int32_t L, const void* q_host, const void* k_host,
                            const void* v_host, void* out_host, uint8_t* keep_host, void* stage_x,
                            void* stage_q, void* stage_k, void* stage_v, void* stage_out,
                            float* logit_dev, uint8_t* keep_dev, void* const* k_caches,
                            void* const* v_caches, int32_t cap, int32_t* cache_len, float scale,
                            void* stream);

/* n_steps decode steps fed from HOST buffers as a pipeline (Eq. 6, once per step): while step t
 * computes, the inputs of step t+1 are copied in and the results of step t-1 are copied out, on
 * two copy streams the context owns (created at the first call, with the events that order them;
 * no device memory is allocated).  Same results as n_steps calls of dl_decode_step_host.
 *   x_host, q_host, k_host, v_host, out_host, keep_host: HOST arrays of n_steps host pointers (the
 *   buffers pinned for full copy speed; keep_host or its entries may be NULL); stage_x dev
 *   [2][B][hidden]; stage_q, stage_k, stage_v, stage_out dev [2][L][B][H][D]; logit_dev dev [2][B];
 *   keep_dev dev [2][B]: two staging sets, used in turn.  The compute runs on `stream`, behind what the
 *   caller queued there; returns after all three streams have been synchronised.  A failed step ends
 *   the sequence: its status is returned once the queued work has drained. */
int32_t dl_decode_steps_host(dl_ctx* ctx, const dl_predictor* p_txt, int32_t n_steps, int32_t B,
                             float threshold, int32_t L, const void* const* x_host,
                             const void* const* q_host, const void* const* k_host,
                             const void* const* v_host, void* const* out_host,
                             uint8_t* const* keep_host, void* stage_x, void* stage_q, void* stage_k,
                             void* stage_v, void* stage_out, float* logit_dev, uint8_t* keep_dev,
                             void* const* k_caches, void* const* v_caches, int32_t cap,
                             int32_t* cache_len, float scale, void* stream);

/* ---- the paper's own predictors (App. "Details of Predictor Architecture") -------------------------------- */

#define DL_PRED2_WIDTH 512      /* width after the input projection; 8 heads of 64; MLP hidden 2048; head 256, 128, 2 */

typedef struct { const void* w; const float* b; } dl_linear;     /* w dev [out][in] bf16, in contiguous; b dev [out] f32 */

/* One pre-norm transformer block over the image tokens of a sequence:
 *   x = x + proj(MHA(LN1(x)));  x = x + fc2(GELU(fc1(LN2(x))))      LayerNorm eps 1e-6, exact-erf GELU,
 * bidirectional scaled-dot-product attention, 8 heads of 64.  ln*_g, ln*_b dev [512] f32; qkv [1536][512] (query,
 * key, value projections stacked, head h owning 64 consecutive outputs of each); proj [512][512]; fc1 [2048][512];
 * fc2 [512][2048]. */
typedef struct {
  const float* ln1_g; const float* ln1_b; dl_linear qkv, proj;
  const float* ln2_g; const float* ln2_b; dl_linear fc1, fc2;
} dl_vit_block;

/* A predictor in the paper's architecture: in [512][hidden]; n_blocks transformer blocks (2 for the image predictor,
 * 0 for the output-text predictor, whose decision depends on the current token alone); head h1 [256][512],
 * h2 [128][256] (GELU after each), w3 dev [2][128] f32, b3 dev [2] f32.  `blocks` is a HOST array. */
typedef struct {
  dl_linear in;
  int32_t n_blocks;
  const dl_vit_block* blocks;
  dl_linear h1, h2;
  const float* w3; const float* b3;
} dl_predictor2;

/* Bytes of scratch dl_predictor2_values needs for `rows` rows (B * n_max).  Negative on bad arguments. */
int64_t dl_predictor2_scratch_bytes(const dl_ctx* ctx, int64_t rows);

/* Decision values of Eq. 5 for every row: D = P(x) in R^{rows x 2}.
 *   x dev [B][n_max][hidden] bf16; n_vis dev [B] or NULL (= n_max): only the first n_vis[b] rows of sequence b are
 *   tokens (they alone attend to one another; padding rows give D = 0, score = -inf, keep = 0);
 *   scratch dev, 256-byte aligned, at least dl_predictor2_scratch_bytes(B * n_max) bytes, caller-owned;
 *   d_out dev [B * n_max][2] f32 or NULL; score_out dev [B * n_max] f32 or NULL: the raw second value D[:,2], the
 *   ranking score of Eq. 11; keep_out dev [B * n_max] or NULL: the argmax of Eq. 5, 1 iff D[:,2] > D[:,1]
 *   (strictly; a NaN drops and records DL_WARN_NAN).  bf16 models only (DL_ERR_UNSUPPORTED otherwise). */
int32_t dl_predictor2_values(dl_ctx* ctx, const dl_predictor2* p, const void* x, const int32_t* n_vis, int32_t B, int32_t n_max,
                      void* scratch, int64_t scratch_bytes, float* d_out, float* score_out, uint8_t* keep_out, void* stream);

/* Eq. 11 with the paper's image predictor: D = P^I(x_vis), then the k[b] tokens with the largest D[:,2] per sequence
 * (ties to the lower index), exactly as dl_prefill_select does with its one-logit predictor. */
int32_t dl_prefill_select2(dl_ctx* ctx, const dl_predictor2* p_img, const void* x_vis, const int32_t* n_vis,
                           const int32_t* k, int32_t B, int32_t n_vis_max, void* scratch, int64_t scratch_bytes,
                           float* d_out, float* score_out, int32_t* kept_idx_out, int32_t k_max, uint8_t* keep_out,
                           void* stream);

/* Eq. 6's decision with the paper's output-text predictor (n_blocks must be 0): keep[b] = D[b][2] > D[b][1].
 *   x_t dev [B][hidden]; d_out dev [B][2] or NULL; keep_out dev [B]. */
int32_t dl_decode_keep2(dl_ctx* ctx, const dl_predictor2* p_txt, const void* x_t, int32_t B, void* scratch,
                        int64_t scratch_bytes, float* d_out, uint8_t* keep_out, void* stream);

/* ---- diagnostics ----------------------------------------------------------------------- */

/* Self-test of the bounded waits (no counterpart in the paper): launches one small kernel that waits, with
 * the library's own wait routine and a bound of `polls` polls (1 .. 65536), on a barrier that can never
 * complete.  The wait gives up, the kernel records DL_ERR_TIMEOUT (detail 0x5e1f) in the status word and
 * returns; nothing traps and the context stays usable.  Asynchronous on `stream`; needs the workspace.
 * dl_device_status then reports the code. */
int32_t dl_selftest_wait_timeout(dl_ctx* ctx, int32_t polls, void* stream);

/* ---- extension, NOT in the paper: K/V cache in 8-bit floating point ---------------------- */

/* Decode attention (Eq. 6) is bound by the bytes of the cache it streams; these two calls store the cache rows as
 * 8-bit floating point in the OCP E4M3 format (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; largest value
 * 448; no infinities) with one fp32 scale per head and tensor:  value = decode(byte) * scale[h].
 * bf16 models with head_dim 128 only (DL_ERR_UNSUPPORTED otherwise). */

/* Rows [0, cache_len[b]) of a bf16 cache as bytes: byte = encode(x / scale[h]), the quotient in fp32, round to
 * nearest with ties to the even code, magnitudes above 448 clamped to 448.  Rows at and past cache_len[b] are not
 * written.
 *   src dev [B][H][cap][128] bf16; scale dev [H] fp32 (> 0); dst dev [B][H][cap][128] uint8 (caller's). */
int32_t dl_quantize_kv_fp8(dl_ctx* ctx, const void* src, const int32_t* cache_len, const float* scale, int32_t B,
                           int32_t cap, void* dst, void* stream);

/* dl_sparse_attn_decode over such caches: the cached rows are read as decode(byte) * scale[h]; the current token is
 * attended with its own bf16 k_t, v_t (kept or not) and, where keep[b] != 0 and the cache has room, appended as
 * bytes at row cache_len[b] (lengths are NOT advanced: dl_commit_len closes the step).
 *   q_t, k_t, v_t, out dev [B][H][128] bf16; k_cache, v_cache dev [B][H][cap][128] uint8, read and (row cache_len[b])
 *   written; k_scale, v_scale dev [H] fp32; keep dev [B] or NULL.  Needs the workspace (split sequences). */
int32_t dl_sparse_attn_decode_fp8(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t, void* k_cache,
                                  void* v_cache, const float* k_scale, const float* v_scale,
                                  const int32_t* cache_len, const uint8_t* keep, int32_t B, int32_t cap, float scale,
                                  void* out, void* stream);

/* The layer stack of a decode step over 8-bit caches (the counterpart of dl_sparse_attn_decode_layers): L launches
 * that overlap on the GPU; with commit != 0 the lengths advance once behind the last layer (cache_len[b] += keep[b]).
 *   q_t, k_t, v_t, out dev [L][B][H][128] bf16; k_caches, v_caches HOST arrays of L dev byte caches [B][H][cap][128];
 *   k_scales, v_scales dev [L][H] fp32; cache_len dev [B], read by every layer, written only with commit. */
int32_t dl_sparse_attn_decode_fp8_layers(dl_ctx* ctx, int32_t L, const void* q_t, const void* k_t, const void* v_t,
                                         void* const* k_caches, void* const* v_caches, const float* k_scales,
                                         const float* v_scales, int32_t* cache_len, const uint8_t* keep, int32_t B,
                                         int32_t cap, float scale, void* out, int32_t commit, void* stream);

/* ---- checked build ---------------------------------------------------------------------- */

/* The library can be built with -DDL_BOUNDS=1 (libdl_sparse_checked.so): every store a kernel makes through an
 * index it computed (cache rows, outputs, partial sums, masks, index lists) is then compared with the extent of its
 * buffer first; an index outside it is NOT used: the store is skipped and DL_ERR_BOUNDS is recorded in the status
 * word with detail = (kernel id << 48) | index.  Nothing traps.  Copies made by the TMA unit are clipped by their
 * tensor maps in either build.  Results are the same as the normal build's; it is slower. */

/* 1 in the checked build, 0 otherwise. */
int32_t dl_build_is_checked(void);

/* Makes one checked store with an index one past the end of a small buffer inside the workspace.  Checked build:
 * the store is skipped, the buffer unchanged, DL_ERR_BOUNDS recorded (kernel id 0x7e, index 64); normal build:
 * DL_ERR_UNSUPPORTED, nothing launched.  Asynchronous on `stream`; needs the workspace. */
int32_t dl_selftest_bounds(dl_ctx* ctx, void* stream);

/* ---- decode attention without any allocation ------------------------------------------- */

/* Size of the library's built-in scratch array (bytes). */
#define DL_STATIC_SCRATCH_BYTES (8u << 20)

/* The paper has no counterpart to this call; it exists for integration reasons only.
 *
 * Same computation, arguments and results as dl_sparse_attn_decode, for callers that must not
 * allocate device memory: code running inside another framework's memory pool or under a fixed
 * memory budget, plugins that are handed their buffers and nothing else, or processes that are
 * already close to the device's capacity and cannot afford a failing cudaMalloc.  Such callers
 * have no workspace to give to dl_set_workspace; here the split partials and arrival tickets
 * live in a fixed array of DL_STATIC_SCRATCH_BYTES that is part of the library image (each GPU
 * that loads the library holds it until the process exits).  The context needs no workspace;
 * without one, device-side conditions (a full cache on append) are skipped silently instead
 * of being recorded.
 *
 *   - Needs  B*H*4 (rounded up to 256) + B*H*(c + 1)*(D+2)*4  bytes of that array, where c is
 *     the largest number of pieces one sequence may be split into: min(cap/64, max(1, W/(B*H)))
 *     with W = 8 warps per SM of the device (16 for fp32 or head_dim 64), or ceil(cap/chunk)
 *     when DL_OPT_DECODE_CHUNK is set.  Large batches are not split (c = 1).  A larger problem
 *     is refused with DL_ERR_WORKSPACE and nothing is launched.
 *   - The first call on a device looks the array's device address up (cudaGetSymbolAddress, with
 *     that device current); make that first call outside any stream capture.
 *   - The call issues one asynchronous memset (the tickets must start at zero; the array keeps
 *     the previous call's contents) and one kernel on `stream`.  It calls no cudaMalloc/cudaFree.
 *   - All calls on a device share the one array: two calls that may overlap on the GPU (different
 *     streams, or different contexts) race on it.  Serialise them on one stream. */
int32_t dl_sparse_attn_decode_static(dl_ctx* ctx, const void* q_t, const void* k_t, const void* v_t,
                                     void* k_cache, void* v_cache, const int32_t* cache_len,
                                     const uint8_t* keep, int32_t B, int32_t cap, float scale, void* out,
                                     void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DL_SPARSE_H_ */
