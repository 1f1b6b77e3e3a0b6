"""CPU oracle for the Dynamic-LLaVA sparsified-inference path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy statement of what the path computes, written from the
paper's equations.  It shares nothing with the CUDA implementation and must never
be imported by the library or its Python binding: only the tests, the smoke check
and the benchmark's CPU-baseline leg use it.

What each function follows
  predictor_logits      Eq. 5 (decision values of the predictor), in the per-token
                        MLP form  s = w2 . GELU(W1 x + b1) + b2  (exact erf GELU)
  k_from_rate           Eq. 11: k = floor(r^I * |S^I|)
  topk_select           Eq. 11: TopkArgmax_k over the predictor score, reduced set in
                        original token order (set builder of Eq. 5)
  decode_keep           Eq. 5 / Eq. 6: keep iff the "keep" value exceeds the "drop" value,
                        i.e. folded single logit > threshold (0), strictly
  nocache_keep          Eq. 12 with the forced last token (decoding without KV cache)
  prefill_keep_mask /   Eq. 5 set builder, Eq. 11 (kept vision rows, then every text row),
  append_rows           Eq. 6 (append K, V of the current token iff its mask is 1)
  attention_masked_full Eq. 7 with diag(G) = 1 under the causal mask: THE definition of
                        attention with dropped tokens
  attention_prefill_compact / attention_decode_compact
                        the same quantity evaluated on the compacted cache (Eq. 1 on the
                        reduced set; Eq. 6: Attention(Q, S^K u K, S^V u V))
  prefill_flops         Eq. 13
  (predictor_paper.py holds the paper's own predictor architectures: App. "Details of Predictor Architecture")

Pins (tests/test_oracle_*.py): closed forms of GELU and of softmax attention,
brute-force sorting, the dense-causal textbook form, masked-vs-compact equality and
the values the paper prints (Tab. 1 token counts and TFLOPs, token-length table).
Task accuracy, perplexity and the paper's wall-clock numbers are parity unpinned:
they need trained weights and datasets that are not available.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

OK = 0
ERR_CAPACITY = -6


# --------------------------------------------------------------------------- predictor
def gelu(h: np.ndarray) -> np.ndarray:
    """GELU(h) = h * Phi(h), Phi the standard normal CDF (exact erf form)."""
    h = np.asarray(h, dtype=np.float64)
    return 0.5 * h * (1.0 + _erf(h / np.sqrt(2.0)))


def predictor_logits(x, w1, b1, w2, b2) -> np.ndarray:
    """Eq. 5, first line, for a per-token MLP predictor with one folded output.

    x [..., d]; w1 [p, d]; b1 [p]; w2 [p]; b2 scalar.  Returns fp64 logits [...]:
    the difference (keep value - drop value) of the two-way decision, which is also
    the ranking score of Eq. 11 when the head has a single output.
    """
    x = np.asarray(x, dtype=np.float64)
    w1 = np.asarray(w1, dtype=np.float64)
    h = x @ w1.T + np.asarray(b1, dtype=np.float64)
    return gelu(h) @ np.asarray(w2, dtype=np.float64) + float(b2)


# --------------------------------------------------------------------------- selection
def k_from_rate(n: int, num: int, den: int) -> int:
    """Eq. 11: floor(r * n) for the rational keep rate r = num / den (integer arithmetic)."""
    return (int(n) * int(num)) // int(den)


def topk_select(score: np.ndarray, k: int):
    """Eq. 11 for one sequence: indices of the k largest scores, larger score first and,
    between equal scores, lower index first; returned in ascending index order together
    with the 0/1 mask M^I.  NaN ranks as -inf; -0.0 equals +0.0."""
    s = np.array(score, dtype=np.float64)
    n = s.shape[0]
    if not 0 <= k <= n:
        raise ValueError("k out of range")
    s[np.isnan(s)] = -np.inf
    # stable sort by descending score: lexsort's last key is primary
    order = np.lexsort((np.arange(n), -s))
    kept = np.sort(order[:k]).astype(np.int32)
    keep = np.zeros(n, dtype=np.uint8)
    keep[kept] = 1
    return kept, keep


def prefill_select(score: np.ndarray, n_vis, k, k_max: int | None = None):
    """Batch form of Eq. 11.  score [B, n_max]; only the first n_vis[b] entries of row b
    are tokens.  Returns kept_idx [B, k_max] (ascending, unused slots -1) and keep [B, n_max]."""
    score = np.asarray(score)
    B, n_max = score.shape
    n_vis = np.full(B, n_max, dtype=np.int64) if n_vis is None else np.asarray(n_vis)
    k = np.asarray(k)
    if k_max is None:
        k_max = int(k.max()) if B else 0
    kept_idx = np.full((B, k_max), -1, dtype=np.int32)
    keep = np.zeros((B, n_max), dtype=np.uint8)
    for b in range(B):
        idx, m = topk_select(score[b, : n_vis[b]], int(k[b]))
        kept_idx[b, : len(idx)] = idx
        keep[b, : n_vis[b]] = m
    return kept_idx, keep


def decode_keep(logit: np.ndarray, threshold: float = 0.0) -> np.ndarray:
    """Eq. 6's mask for the current token: 1 iff logit > threshold (strict; NaN drops)."""
    logit = np.asarray(logit, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        return (logit > threshold).astype(np.uint8)


def nocache_keep(logit: np.ndarray, n_gen, threshold: float = 0.0) -> np.ndarray:
    """Decoding WITHOUT KV cache (Eq. 12, and the sentence above Eq. 6): the mask of all generated
    tokens at once, M^OT = [logit > threshold], except that the last generated token of every
    sequence is always kept (it produces the next token).  logit [B, n_max]; n_gen [B] valid
    tokens per sequence (None = all); slots past n_gen[b] are 0."""
    logit = np.asarray(logit, dtype=np.float64)
    B, n_max = logit.shape
    n_gen = np.full(B, n_max, dtype=np.int64) if n_gen is None else np.asarray(n_gen)
    keep = np.zeros((B, n_max), dtype=np.uint8)
    for b in range(B):
        n = int(n_gen[b])
        keep[b, :n] = decode_keep(logit[b, :n], threshold)
        if n > 0:
            keep[b, n - 1] = 1
    return keep


# --------------------------------------------------------------------------- compaction
def append_rows(k_src, v_src, keep, t_src, k_cache, v_cache, cache_len, commit: bool = True):
    """Append, in token order, the rows of k_src / v_src whose mask is 1 (Eq. 5 set builder;
    Eq. 6 when there is one source row per sequence).

    k_src, v_src [B, T, H, D] (any dtype: rows are copied bit for bit); keep [B, T] or None
    (= keep all); t_src [B] valid source rows or None (= T); caches [B, H, cap, D];
    cache_len [B] int, advanced in place when `commit`.  A sequence whose kept rows do
    not fit is left untouched and reported: returns (status, per-sequence appended count).
    """
    B, T, H, D = k_src.shape
    cap = k_cache.shape[2]
    status = OK
    counts = np.zeros(B, dtype=np.int32)
    for b in range(B):
        tb = T if t_src is None else int(t_src[b])
        rows = [t for t in range(tb) if keep is None or keep[b, t] != 0]
        if cache_len[b] + len(rows) > cap:
            status = ERR_CAPACITY
            continue
        pos = int(cache_len[b])
        for t in rows:
            for h in range(H):
                k_cache[b, h, pos, :] = k_src[b, t, h, :]
                v_cache[b, h, pos, :] = v_src[b, t, h, :]
            pos += 1
        counts[b] = len(rows)
        if commit:
            cache_len[b] = pos
    return status, counts


def prefill_keep_mask(keep_vis: np.ndarray, n_vis, n_text) -> np.ndarray:
    """Full prefill mask M = M^I u {1}^{N_T} (Sec. 3.3.3) laid out as [B, n_vis_max + n_text_max]
    for sources that store the vision rows first and the text rows right after them."""
    B, nv = keep_vis.shape
    n_text = np.asarray(n_text)
    out = np.zeros((B, nv + int(n_text.max())), dtype=np.uint8)
    for b in range(B):
        out[b, :nv] = keep_vis[b]
        out[b, nv: nv + int(n_text[b])] = 1
    return out


# --------------------------------------------------------------------------- attention
def _softmax_rows(z: np.ndarray, visible: np.ndarray) -> np.ndarray:
    """Eq. 7: exp(z_ij) G_ij / sum_k exp(z_ik) G_ik, evaluated with the row maximum
    subtracted (the quotient is unchanged)."""
    zz = np.where(visible, z, -np.inf)
    m = zz.max(axis=-1, keepdims=True)
    e = np.where(visible, np.exp(zz - m), 0.0)
    return e / e.sum(axis=-1, keepdims=True)


def attention_masked_full(q, k, v, mask, scale: float) -> np.ndarray:
    """Definition of attention under a token mask (Eq. 7 with diag(G) = 1, causal).

    One head: q, k, v [N, D] over the FULL, uncompacted context; mask [N] in {0,1}.
    Row i sees column j iff j <= i and (mask[j] == 1 or j == i).  Returns [N, D]
    (rows of dropped tokens are what such a token computes in its own step)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n = q.shape[0]
    g = np.broadcast_to(np.asarray(mask).astype(bool)[None, :], (n, n)).copy()
    np.fill_diagonal(g, True)
    causal = np.tril(np.ones((n, n), dtype=bool))
    p = _softmax_rows((q @ k.T) * scale, g & causal)
    return p @ v


def attention_prefill_compact(q_c, k_c, v_c, n: int, scale: float) -> np.ndarray:
    """Eq. 1 on the reduced set: causal attention of the first n compact rows against
    themselves.  One head: q_c, k_c, v_c [>= n, D]; returns [n, D]."""
    q = np.asarray(q_c[:n], dtype=np.float64)
    k = np.asarray(k_c[:n], dtype=np.float64)
    v = np.asarray(v_c[:n], dtype=np.float64)
    out = np.zeros((n, q.shape[1]))
    for i in range(n):
        z = (k[: i + 1] @ q[i]) * scale
        e = np.exp(z - z.max())
        out[i] = (e / e.sum()) @ v[: i + 1]
    return out


def attention_decode_compact(q_t, k_t, v_t, k_cache, v_cache, n: int, scale: float) -> np.ndarray:
    """Eq. 6, second line: Attention(Q, S^K u K, S^V u V) for one head and one token.
    q_t, k_t, v_t [D]; caches [>= n, D] of which the first n rows are valid.  The current
    token's own K/V always take part, whether or not it is kept afterwards."""
    q = np.asarray(q_t, dtype=np.float64)
    d = q.shape[0]
    k = np.vstack([np.asarray(k_cache[:n], dtype=np.float64).reshape(n, d),
                   np.asarray(k_t, dtype=np.float64)[None, :]])
    v = np.vstack([np.asarray(v_cache[:n], dtype=np.float64).reshape(n, d),
                   np.asarray(v_t, dtype=np.float64)[None, :]])
    z = (k @ q) * scale
    e = np.exp(z - z.max())
    return (e / e.sum()) @ v


# --------------------------------------------------------------------------- accounting
def prefill_flops(batch: int, n_tokens: int, width: int) -> int:
    """Eq. 13: FLOPs of one decoder layer over n_tokens image tokens."""
    return 32 * batch * n_tokens * width ** 2 + 4 * batch * n_tokens ** 2 * width


def prefill_flops_model(n_layers: int, dense_layers: int, n_full: int, n_kept: int, width: int,
                        batch: int = 1) -> int:
    """Eq. 13 summed over a model whose first `dense_layers` layers see all n_full image
    tokens and whose remaining layers see n_kept (the decision is taken once, after layer l)."""
    return (dense_layers * prefill_flops(batch, n_full, width)
            + (n_layers - dense_layers) * prefill_flops(batch, n_kept, width))
