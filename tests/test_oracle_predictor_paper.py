"""Pins of the oracle for the paper's own predictors (App. "Details of Predictor Architecture"; Eq. 5 argmax,
Eq. 11 ranking by the second decision value): closed forms, a separately written loop form, special weights
that reduce a part to something known, and invariances that a wrong index or a dropped term would break."""
import numpy as np
import pytest

from oracle import dl_oracle as orc
from oracle import predictor_paper as pp
from paper_2412_00876_b200 import workloads as wl


def _small_cfg():
    return wl.CONFIGS[1].scaled(hidden=64)


def _params(which="img", width=32, mlp=48, hidden=24, seed=0):
    """Tiny random parameters with the architecture's structure (4 heads of 8 on width 32)."""
    rng = np.random.default_rng(seed)
    r = lambda *s: rng.normal(size=s)
    blk = lambda: {"ln1_g": 1 + 0.1 * r(width), "ln1_b": 0.1 * r(width), "w_qkv": r(3 * width, width) / 6,
                   "b_qkv": 0.1 * r(3 * width), "w_o": r(width, width) / 6, "b_o": 0.1 * r(width),
                   "ln2_g": 1 + 0.1 * r(width), "ln2_b": 0.1 * r(width), "w_fc1": r(mlp, width) / 6,
                   "b_fc1": 0.1 * r(mlp), "w_fc2": r(width, mlp) / 7, "b_fc2": 0.1 * r(width)}
    return {"w_in": r(width, hidden) / 5, "b_in": 0.1 * r(width), "blocks": [blk(), blk()] if which == "img" else [],
            "head": {"w1": r(16, width) / 6, "b1": 0.1 * r(16), "w2": r(8, 16) / 4, "b2": 0.1 * r(8),
                     "w3": r(2, 8) / 3, "b3": 0.1 * r(2)}}


def test_layer_norm_closed_forms():
    g, b = np.array([2.0, 3.0, 4.0, 5.0]), np.array([0.5, -1.0, 0.0, 7.0])
    assert np.allclose(pp.layer_norm(np.full((3, 4), 9.25), g, b), b)            # a constant row: only the shift is left
    x = np.array([[1.0, -1.0, 1.0, -1.0]])                                          # mean 0, variance 1
    assert np.allclose(pp.layer_norm(x, g, b, eps=0.0), x * g + b)
    y = pp.layer_norm(np.random.default_rng(0).normal(size=(5, 64)) * 7 + 3, 1.0, 0.0, eps=0.0)
    assert np.allclose(y.mean(axis=1), 0) and np.allclose((y ** 2).mean(axis=1), 1)
    x = np.random.default_rng(1).normal(size=(2, 16))
    assert np.allclose(pp.layer_norm(3 * x + 11, 1.0, 0.0, eps=0.0), pp.layer_norm(x, 1.0, 0.0, eps=0.0))   # shift and scale


def _mha_loops(x, w_qkv, b_qkv, w_o, b_o, H):
    """Multi-head attention written out with explicit loops over heads, rows and keys."""
    n, c = x.shape
    hd = c // H
    q = np.zeros((n, c)); k = np.zeros((n, c)); v = np.zeros((n, c))
    for i in range(n):
        for o in range(c):
            q[i, o] = sum(w_qkv[o, j] * x[i, j] for j in range(c)) + b_qkv[o]
            k[i, o] = sum(w_qkv[c + o, j] * x[i, j] for j in range(c)) + b_qkv[c + o]
            v[i, o] = sum(w_qkv[2 * c + o, j] * x[i, j] for j in range(c)) + b_qkv[2 * c + o]
    att = np.zeros((n, c))
    for h in range(H):
        for i in range(n):
            z = [sum(q[i, h * hd + d] * k[j, h * hd + d] for d in range(hd)) / np.sqrt(hd) for j in range(n)]
            e = [np.exp(t - max(z)) for t in z]
            for d in range(hd):
                att[i, h * hd + d] = sum(e[j] * v[j, h * hd + d] for j in range(n)) / sum(e)
    return np.array([[sum(w_o[o, j] * att[i, j] for j in range(c)) + b_o[o] for o in range(c)] for i in range(n)])


def test_multi_head_attention_equals_the_loop_form():
    rng = np.random.default_rng(2)
    n, c, H = 5, 8, 2
    x, w_qkv, b_qkv = rng.normal(size=(n, c)), rng.normal(size=(3 * c, c)), rng.normal(size=3 * c)
    w_o, b_o = rng.normal(size=(c, c)), rng.normal(size=c)
    assert np.allclose(pp.multi_head_attention(x, w_qkv, b_qkv, w_o, b_o, H), _mha_loops(x, w_qkv, b_qkv, w_o, b_o, H))


def test_attention_with_zero_queries_is_the_mean_of_the_values():
    rng = np.random.default_rng(3)
    n, c, H = 7, 8, 2
    x = rng.normal(size=(n, c))
    w_qkv = rng.normal(size=(3 * c, c)); b_qkv = rng.normal(size=3 * c)
    w_qkv[:c] = 0; b_qkv[:c] = 0                                     # q = 0: every score 0, uniform weights
    v = x @ w_qkv[2 * c:].T + b_qkv[2 * c:]
    out = pp.multi_head_attention(x, w_qkv, b_qkv, np.eye(c), np.zeros(c), H)
    assert np.allclose(out, np.broadcast_to(v.mean(axis=0), (n, c)))


def test_block_with_zero_output_projections_is_the_identity():
    p = _params()
    blk = p["blocks"][0]
    blk["w_o"][:] = 0; blk["b_o"][:] = 0; blk["w_fc2"][:] = 0; blk["b_fc2"][:] = 0
    x = np.random.default_rng(4).normal(size=(6, 32))
    assert np.array_equal(pp.vit_block(x, blk, 4), x)
    blk["b_fc2"][:] = 0.25                                            # only the second residual branch's bias
    assert np.allclose(pp.vit_block(x, blk, 4), x + 0.25)


def test_image_predictor_is_equivariant_to_token_order_and_blind_to_padding():
    """No positional term and no causal mask: permuting the image tokens permutes the decisions; rows past
    n_vis take no part (a sequence gives the same decisions alone or padded in a batch)."""
    p = _params()                                                     # width 32: 8 heads of 4
    rng = np.random.default_rng(5)
    x = rng.normal(size=(1, 9, 24))
    D = pp.image_predictor(x, p)
    perm = rng.permutation(9)
    assert np.allclose(pp.image_predictor(x[:, perm], p)[0], D[0, perm])
    xb = np.concatenate([x, rng.normal(size=(1, 9, 24))], axis=0)
    xb[0, 6:] = 1e6                                                   # hostile padding
    Db = pp.image_predictor(xb, p, n_vis=[6, 9])
    assert np.allclose(Db[0, :6], pp.image_predictor(x[:, :6], p)[0]) and np.all(Db[0, 6:] == 0)
    # ... and the tokens DO see one another: changing one token changes the others' decisions
    x2 = x.copy(); x2[0, 0] += 1.0
    assert np.abs(pp.image_predictor(x2, p)[0, 1:] - D[0, 1:]).max() > 1e-6


def test_text_predictor_is_token_wise_and_equals_the_written_out_chain():
    p = _params("txt")
    rng = np.random.default_rng(6)
    x = rng.normal(size=(4, 3, 24))
    D = pp.text_predictor(x, p)
    assert D.shape == (4, 3, 2)
    for b in range(4):
        for t in range(3):
            h = p["w_in"] @ x[b, t] + p["b_in"]
            h = orc.gelu(p["head"]["w1"] @ h + p["head"]["b1"])
            h = orc.gelu(p["head"]["w2"] @ h + p["head"]["b2"])
            assert np.allclose(D[b, t], p["head"]["w3"] @ h + p["head"]["b3"])
    x2 = x.copy(); x2[0, 0] += 1.0                                    # another token changes nothing here
    assert np.array_equal(pp.text_predictor(x2, p)[1:], D[1:]) and np.array_equal(pp.text_predictor(x2, p)[0, 1:], D[0, 1:])


def test_two_way_head_with_a_constant_first_output_is_the_one_logit_decision():
    """W3[0] = 0 makes D1 = b3[0] for every token: keep iff D2 > b3[0], i.e. dl_oracle.decode_keep of the folded
    logit D2 - D1 with threshold 0; and ranking by D2 equals ranking by the folded logit."""
    p = _params("txt")
    p["head"]["w3"][0] = 0
    x = np.random.default_rng(7).normal(size=(50, 24))
    D = pp.text_predictor(x, p)
    assert np.allclose(D[:, 0], p["head"]["b3"][0])
    folded = D[:, 1] - D[:, 0]
    assert np.array_equal(pp.decision_keep(D), orc.decode_keep(folded))
    assert np.array_equal(orc.topk_select(pp.ranking_score(D), 10)[0], orc.topk_select(folded, 10)[0])
    # in general the ranking value and the keep test are different quantities
    p2 = _params("txt", seed=8)
    D2 = pp.text_predictor(x, p2)
    assert not np.array_equal(orc.topk_select(D2[:, 1], 10)[0], orc.topk_select(D2[:, 1] - D2[:, 0], 10)[0])
    assert list(pp.decision_keep(np.array([[0.0, 0.0], [1.0, 2.0], [2.0, 1.0], [np.nan, 1.0]]))) == [0, 1, 0, 0]


def test_seeded_weights_have_the_papers_shapes():
    cfg = wl.CONFIGS[2]
    pi, pt = wl.make_predictor_paper(cfg, "img"), wl.make_predictor_paper(cfg, "txt")
    assert pi["w_in"].shape == (512, cfg.hidden) and len(pi["blocks"]) == 2 and len(pt["blocks"]) == 0
    b = pi["blocks"][0]
    assert b["w_qkv"].shape == (1536, 512) and b["w_fc1"].shape == (2048, 512) and b["w_fc2"].shape == (512, 2048)
    h = pi["head"]
    assert h["w1"].shape == (256, 512) and h["w2"].shape == (128, 256) and h["w3"].shape == (2, 128)
    D = pp.text_predictor(wl.host_normal(cfg, wl.S_X_TXT, (64, cfg.hidden)), pt)
    assert 0.1 < np.abs(D).mean() < 10 and 5 < pp.decision_keep(D).sum() < 59      # decisions of both kinds
