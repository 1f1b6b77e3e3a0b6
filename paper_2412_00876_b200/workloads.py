"""Seeded synthetic inputs shaped like the Dynamic-LLaVA inference workloads.

This module only *draws numbers and describes shapes*.  It contains none of the
method's arithmetic (no predictor, no selection, no compaction, no attention),
so that the CUDA path and the CPU oracle can both be fed from it without
sharing any logic.

Shapes follow LLaVA-1.5 as used in the paper (576 vision tokens per image,
hidden 4096 / 5120, 32 / 40 heads of 128; Sec. 4.1 and the token-length table
of the appendix); value distributions are i.i.d. normals because trained
weights and the paper's datasets are not available.

Host tensors come from numpy's Philox counter-based generator keyed by
(config id, stream id).  Large device tensors (activations and K/V for the
batched configurations) are drawn on the device by a seeded torch generator;
tests copy the slices they need back to the host, so both sides always see
the same bytes.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 0x24120876

# stream ids (one independent random stream per tensor kind)
S_X_VIS, S_W1_IMG, S_W2_IMG, S_W1_TXT, S_W2_TXT = 0, 1, 2, 3, 4
S_Q, S_K, S_V, S_X_TXT, S_LEN, S_DEC_Q, S_DEC_K, S_DEC_V, S_CACHE_K, S_CACHE_V, S_LOGIT = (
    5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15)


@dataclass(frozen=True)
class Config:
    """One synthetic workload (shapes only)."""
    cid: int            # 1-based id, used in the seed
    name: str
    dtype: str          # "f32" or "bf16": storage type of activations, K/V and W1
    B: int              # sequences per batch
    hidden: int         # d
    n_heads: int        # H
    head_dim: int       # D
    n_layers: int       # L: layers after the decision layer (all of them compacted)
    n_vis: int          # N_I vision tokens per sequence
    k_vis: int          # kept vision tokens per sequence
    n_text: int         # N_T prompt text tokens
    n_gen: int          # N_OT generated tokens
    keep_rate: float    # target fraction of generated tokens kept
    pred_hidden: int    # width of the predictor's hidden layer

    @property
    def n0(self) -> int:
        """Compact prefill length k + N_T."""
        return self.k_vis + self.n_text

    @property
    def cap(self) -> int:
        """Rows allocated per (sequence, head) cache: every token could be kept."""
        return (self.n0 + self.n_gen + 63) // 64 * 64

    @property
    def elt_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def scaled(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    1: Config(1, "toy-fp32", "f32", 1, 512, 8, 64, 1, 144, 36, 32, 64, 0.5, 128),
    2: Config(2, "llava1.5-7b-1layer", "bf16", 1, 4096, 32, 128, 1, 576, 144, 64, 256, 0.5, 1024),
    3: Config(3, "decode-serving-7b-b32-l32", "bf16", 32, 4096, 32, 128, 32, 576, 144, 128, 1024, 0.5, 1024),
    4: Config(4, "llava1.5-13b-b64-l40", "bf16", 64, 5120, 40, 128, 40, 576, 144, 96, 512, 0.5, 1280),
    5: Config(5, "multicrop-7b-b16-l32", "bf16", 16, 4096, 32, 128, 32, 2880, 576, 256, 2048, 0.4, 1024),
}


# --------------------------------------------------------------------------
# storage-type rounding (bf16 has no numpy dtype: carried as uint16 bit patterns)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array whose values are exactly representable in the storage type."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def storage_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """Raw storage of a (storage-exact) float32 array: float32 itself or uint16 bf16 bits."""
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    return f32_to_bf16_bits(x)


def bits_to_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    """Exact float64 value of stored elements (what the oracle computes on)."""
    if dtype == "f32":
        return np.asarray(bits, dtype=np.float32).astype(np.float64)
    return bf16_bits_to_f32(bits).astype(np.float64)


# --------------------------------------------------------------------------
# host generators
# --------------------------------------------------------------------------
def host_rng(cfg_id: int, stream: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[BASE_SEED + 1000 * cfg_id + stream, sub]))


def host_normal(cfg: Config, stream: int, shape, std: float = 1.0, dtype: str | None = None,
                sub: int = 0) -> np.ndarray:
    """N(0, std^2) draws, rounded to the storage type; returned as float32."""
    x = host_rng(cfg.cid, stream, sub).standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    return round_to_storage(x, dtype or cfg.dtype)


_BIAS_TABLE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "workload_bias.json")


def stored_bias(cfg: Config, which: str) -> float:
    """Second-layer bias b2 that centres the predictor's logits for `which` in {"img","txt"}.

    The values were fixed once by a seeded calibration draw (see the script beside the
    oracle that writes the table) so that about `keep_rate` of N(0,1) rows get a
    positive logit; they are plain inputs to both implementations.
    """
    with open(_BIAS_TABLE) as f:
        tab = json.load(f)
    return float(tab[f"{cfg.cid}:{which}:{cfg.hidden}:{cfg.pred_hidden}"])


@dataclass
class Predictor:
    """Weights of one token predictor: score = w2 . GELU(W1 x + b1) + b2."""
    w1: np.ndarray   # [pred_hidden, hidden] float32 values exact in the storage type
    b1: np.ndarray   # [pred_hidden] float32
    w2: np.ndarray   # [pred_hidden] float32
    b2: float


def make_predictor(cfg: Config, which: str, b2: float | None = None) -> Predictor:
    s1, s2 = (S_W1_IMG, S_W2_IMG) if which == "img" else (S_W1_TXT, S_W2_TXT)
    w1 = host_normal(cfg, s1, (cfg.pred_hidden, cfg.hidden), std=0.02)
    w2 = host_normal(cfg, s2, (cfg.pred_hidden,), std=0.02, dtype="f32")
    # a small non-zero first-layer bias so that a dropped or mis-indexed b1 is visible
    b1 = host_normal(cfg, s2, (cfg.pred_hidden,), std=0.02, dtype="f32", sub=1)
    if b2 is None:
        b2 = stored_bias(cfg, which)
    return Predictor(w1, b1, w2, float(np.float32(b2)))


S_PAPER_PRED = 40       # streams 40.. : weights of the paper's own predictors


def make_predictor_paper(cfg: Config, which: str, width: int = 512, n_blocks: int = 2, mlp_hidden: int = 2048,
                         out_bias: float = 0.0) -> dict:
    """Seeded weights of the paper's predictor architecture (linear d -> 512; two transformer blocks for the
    image predictor; head 512 -> 256 -> 128 -> 2).  Matrices ~ N(0, 1/fan_in), rounded to the storage type;
    biases and LayerNorm parameters in float32 (scales near 1).  `which` in {"img", "txt"}; the text predictor
    has no blocks.  out_bias is added to the second output's bias (moves the keep rate)."""
    base = S_PAPER_PRED + (0 if which == "img" else 20)
    n = [0]

    def mat(o, i):
        n[0] += 1
        return host_normal(cfg, base, (o, i), std=1.0 / np.sqrt(i), sub=n[0])

    def vec(o, std=0.1, mean=0.0):
        n[0] += 1
        return (host_normal(cfg, base, (o,), std=std, dtype="f32", sub=n[0]) + np.float32(mean)).astype(np.float32)

    p = {"w_in": mat(width, cfg.hidden), "b_in": vec(width), "blocks": []}
    for _ in range(n_blocks if which == "img" else 0):
        p["blocks"].append({"ln1_g": vec(width, 0.1, 1.0), "ln1_b": vec(width), "w_qkv": mat(3 * width, width),
                            "b_qkv": vec(3 * width), "w_o": mat(width, width), "b_o": vec(width),
                            "ln2_g": vec(width, 0.1, 1.0), "ln2_b": vec(width), "w_fc1": mat(mlp_hidden, width),
                            "b_fc1": vec(mlp_hidden), "w_fc2": mat(width, mlp_hidden), "b_fc2": vec(width)})
    b3 = vec(2)
    b3[1] += np.float32(out_bias)
    p["head"] = {"w1": mat(256, width), "b1": vec(256), "w2": mat(128, 256), "b2": vec(128),
                 "w3": host_normal(cfg, base, (2, 128), std=1.0 / np.sqrt(128), dtype="f32", sub=99), "b3": b3}
    return p


def ragged_text_lengths(cfg: Config) -> np.ndarray:
    """Per-sequence prompt lengths, uniform in [N_T/2, N_T] (correctness variant)."""
    lo = max(1, cfg.n_text // 2)
    return host_rng(cfg.cid, S_LEN).integers(lo, cfg.n_text + 1, size=cfg.B).astype(np.int32)


def static_keep_pattern(kind: str, n: int, cfg: Config | None = None) -> np.ndarray:
    """The paper's two static sparsifiers, as uint8 masks: "structure" drops every
    other token; "random" keeps each token with probability 1/2 (Tab. 3 discussion)."""
    if kind == "structure":
        return (np.arange(n) % 2 == 0).astype(np.uint8)
    if kind == "random":
        cid = cfg.cid if cfg else 0
        return (host_rng(cid, S_LOGIT, 7).random(n) < 0.5).astype(np.uint8)
    raise ValueError(kind)


# --------------------------------------------------------------------------
# device generators (torch is imported lazily: the oracle's tests do not need it)
# --------------------------------------------------------------------------
def torch_dtype(dtype: str):
    import torch
    return torch.float32 if dtype == "f32" else torch.bfloat16


def to_torch(x_f32: np.ndarray, dtype: str, device="cpu"):
    """Storage-exact float32 numpy array -> torch tensor of the storage type."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32))
    return t.to(device=device, dtype=torch_dtype(dtype))


def from_torch(t) -> np.ndarray:
    """torch tensor (any float type) -> float64 numpy array, exact."""
    return t.detach().to("cpu").double().numpy()


def device_normal(cfg: Config, stream: int, shape, device, std: float = 1.0, dtype: str | None = None,
                  sub: int = 0):
    """N(0, std^2) draws made on `device` by a seeded torch generator, in the storage type."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((BASE_SEED + 1000 * cfg.cid + stream) * 65537 + sub)
    out = torch.empty(shape, device=device, dtype=torch_dtype(dtype or cfg.dtype))
    out.normal_(0.0, std, generator=g)
    return out
