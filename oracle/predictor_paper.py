"""CPU oracle for the paper's own predictors.  TEST INFRASTRUCTURE ONLY (see dl_oracle.py).

App. "Details of Predictor Architecture": both predictors first reduce the model width d to 512 with a
linear layer; the image predictor then applies two vision-transformer blocks over the image tokens of a
sequence and a three-layer MLP 512 -> 256 -> 128 -> 2; the output-text predictor is the same without the
transformer blocks, so that its decision depends on the current token alone.  The two outputs per token are
the decision values D of Eq. 5: the token is kept iff the second value exceeds the first (argmax), and the
prefill ranking of Eq. 11 uses the raw second value D[:, 2].

What the paper leaves open (its figure of the predictors is missing) is read as follows, and written in
fp64 numpy with no blocking or fusion:
  * transformer block = the pre-norm block of the cited vision transformers:
        x = x + Proj(MHA(LN(x)));  x = x + FC2(GELU(FC1(LN(x))))
    with 8 heads of 64 dimensions, scaled dot-product attention among ALL image tokens of the sequence
    (no causal mask, no positional term: the tokens come out of a decoder layer), hidden width 4 x 512,
    LayerNorm with eps = 1e-6, exact-erf GELU, biases everywhere;
  * MLP head = Linear, GELU, Linear, GELU, Linear; no softmax on the two outputs (the argmax and the
    ranking by the second value are taken on the raw values);
  * no normalisation after the last block.

Pins (tests/test_oracle_predictor_paper.py): LayerNorm closed forms, a separately written loop form of
multi-head attention, blocks with zero output projections (identity), zero query weights (attention = mean
of the values), the head with a constant first output (reduces to the one-logit decision of dl_oracle),
permutation equivariance over the image tokens, and that the text predictor is token-wise.
"""
from __future__ import annotations

import numpy as np

from .dl_oracle import gelu

WIDTH, HEADS, HEAD_DIM, MLP_HIDDEN, EPS = 512, 8, 64, 2048, 1e-6


def linear(x, w, b):
    """y = x W^T + b with W [out, in]."""
    return np.asarray(x, np.float64) @ np.asarray(w, np.float64).T + np.asarray(b, np.float64)


def layer_norm(x, gamma, beta, eps: float = EPS):
    """(x - mean) / sqrt(var + eps) * gamma + beta over the last dimension (biased variance)."""
    x = np.asarray(x, np.float64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * np.asarray(gamma, np.float64) + np.asarray(beta, np.float64)


def multi_head_attention(x, w_qkv, b_qkv, w_o, b_o, n_heads: int = HEADS):
    """Bidirectional multi-head self-attention over the rows of x [n, c].  w_qkv [3c, c] stacks the query, key
    and value projections (head h owns columns h*c/H .. of each); scores are scaled by 1/sqrt(c/H)."""
    x = np.asarray(x, np.float64)
    n, c = x.shape
    hd = c // n_heads
    qkv = linear(x, w_qkv, b_qkv)
    q, k, v = qkv[:, :c], qkv[:, c: 2 * c], qkv[:, 2 * c:]
    out = np.zeros((n, c))
    for h in range(n_heads):
        sl = slice(h * hd, (h + 1) * hd)
        z = (q[:, sl] @ k[:, sl].T) / np.sqrt(hd)
        p = np.exp(z - z.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        out[:, sl] = p @ v[:, sl]
    return linear(out, w_o, b_o)


def vit_block(x, blk: dict, n_heads: int = HEADS):
    """One pre-norm transformer block over the image tokens of ONE sequence, x [n, 512]."""
    x = np.asarray(x, np.float64)
    x = x + multi_head_attention(layer_norm(x, blk["ln1_g"], blk["ln1_b"]), blk["w_qkv"], blk["b_qkv"],
                                 blk["w_o"], blk["b_o"], n_heads)
    h = gelu(linear(layer_norm(x, blk["ln2_g"], blk["ln2_b"]), blk["w_fc1"], blk["b_fc1"]))
    return x + linear(h, blk["w_fc2"], blk["b_fc2"])


def mlp_head(x, hp: dict):
    """512 -> 256 -> 128 -> 2, GELU after the first two layers.  Returns D [..., 2]."""
    h = gelu(linear(x, hp["w1"], hp["b1"]))
    h = gelu(linear(h, hp["w2"], hp["b2"]))
    return linear(h, hp["w3"], hp["b3"])


def text_predictor(x, params: dict):
    """P^OT: x [..., d] -> D [..., 2], every token on its own (Eq. 6 decides on the current token only)."""
    return mlp_head(linear(x, params["w_in"], params["b_in"]), params["head"])


def image_predictor(x_vis, params: dict, n_vis=None):
    """P^I for a batch: x_vis [B, n_max, d]; only the first n_vis[b] rows of sequence b are image tokens and
    attend to one another.  Returns D [B, n_max, 2] (rows past n_vis[b] are 0)."""
    x_vis = np.asarray(x_vis, np.float64)
    B, n_max, _ = x_vis.shape
    n_vis = np.full(B, n_max) if n_vis is None else np.asarray(n_vis)
    out = np.zeros((B, n_max, 2))
    for b in range(B):
        n = int(n_vis[b])
        if n == 0:
            continue
        t = linear(x_vis[b, :n], params["w_in"], params["b_in"])
        for blk in params["blocks"]:
            t = vit_block(t, blk)
        out[b, :n] = mlp_head(t, params["head"])
    return out


def decision_keep(D) -> np.ndarray:
    """Eq. 5: M = argmax_j D: 1 iff the second value is greater than the first (strictly; NaN drops)."""
    D = np.asarray(D, np.float64)
    with np.errstate(invalid="ignore"):
        return (D[..., 1] > D[..., 0]).astype(np.uint8)


def ranking_score(D) -> np.ndarray:
    """Eq. 11: the predictor score of a token is the raw second decision value D[:, 2]."""
    return np.asarray(D, np.float64)[..., 1]
