"""Pins for the oracle's predictor (Eq. 5 in per-token MLP form) and for k = floor(r N)."""
import json
import math
import os

import numpy as np

from oracle import dl_oracle as orc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def phi(x):  # standard normal CDF from the C library's erf
    return 0.5 * (1.0 + math.erf(x / math.sqrt(2.0)))


def test_gelu_closed_forms():
    assert orc.gelu(np.array([0.0]))[0] == 0.0
    # GELU(1) = Phi(1); Phi(1) = 0.841344746068543 (standard normal table)
    assert abs(orc.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    x = np.linspace(-6, 6, 241)
    g = orc.gelu(x)
    # Phi(x) + Phi(-x) = 1  =>  GELU(x) - GELU(-x) = x
    assert np.allclose(g - orc.gelu(-x), x, atol=1e-14)
    # large |x|: identity on the right, zero on the left
    assert abs(orc.gelu(np.array([40.0]))[0] - 40.0) < 1e-12
    assert abs(orc.gelu(np.array([-40.0]))[0]) < 1e-12
    for xi, gi in zip(x, g):
        assert abs(gi - xi * phi(xi)) < 1e-14
    # the tanh approximation is a different function: the oracle must not be it
    t = 0.5 * 1.5 * (1 + math.tanh(math.sqrt(2 / math.pi) * (1.5 + 0.044715 * 1.5 ** 3)))
    assert abs(orc.gelu(np.array([1.5]))[0] - t) > 1e-5


def test_zero_first_layer_reduces_to_bias_terms():
    rng = np.random.default_rng(1)
    p, d = 7, 5
    b1, w2, b2 = rng.normal(size=p), rng.normal(size=p), 0.37
    s = orc.predictor_logits(rng.normal(size=(3, d)), np.zeros((p, d)), b1, w2, b2)
    expect = sum(w2[j] * b1[j] * phi(b1[j]) for j in range(p)) + b2
    assert np.allclose(s, expect, atol=1e-14)


def test_one_hot_rows_pick_inputs():
    rng = np.random.default_rng(2)
    d, p = 6, 4
    perm = [4, 0, 5, 2]
    w1 = np.zeros((p, d))
    for j, i in enumerate(perm):
        w1[j, i] = 1.0
    x = rng.normal(size=(5, d))
    b1, w2 = rng.normal(size=p), rng.normal(size=p)
    s = orc.predictor_logits(x, w1, b1, w2, -0.25)
    for r in range(5):
        e = sum(w2[j] * (x[r, perm[j]] + b1[j]) * phi(x[r, perm[j]] + b1[j]) for j in range(p)) - 0.25
        assert abs(s[r] - e) < 1e-13


def test_brute_force_loops_non_square():
    """Triple loop over a non-square W1 catches a transposed operand or a dropped bias."""
    rng = np.random.default_rng(3)
    n, d, p = 4, 9, 3
    x, w1 = rng.normal(size=(n, d)), rng.normal(size=(p, d))
    b1, w2, b2 = rng.normal(size=p), rng.normal(size=p), 1.25
    s = orc.predictor_logits(x, w1, b1, w2, b2)
    for r in range(n):
        acc = b2
        for j in range(p):
            h = b1[j]
            for i in range(d):
                h += w1[j, i] * x[r, i]
            acc += w2[j] * h * phi(h)
        assert abs(s[r] - acc) < 1e-12


def test_linear_in_second_layer_and_bias_shift():
    rng = np.random.default_rng(4)
    x, w1, b1 = rng.normal(size=(8, 10)), rng.normal(size=(6, 10)), rng.normal(size=6)
    wa, wb = rng.normal(size=6), rng.normal(size=6)
    sa = orc.predictor_logits(x, w1, b1, wa, 0.0)
    sb = orc.predictor_logits(x, w1, b1, wb, 0.0)
    sab = orc.predictor_logits(x, w1, b1, 2 * wa - 3 * wb, 0.5)
    assert np.allclose(sab, 2 * sa - 3 * sb + 0.5, atol=1e-12)


def test_k_is_floor_of_rate_times_n_paper_value():
    g = GOLD["kept_vision_tokens"]
    assert orc.k_from_rate(g["n"], g["rate_num"], g["rate_den"]) == g["k"]  # 115, not 116
    assert orc.k_from_rate(2880, 20, 100) == 576   # 0.2 * 2880 in floating point is 576.0000000000001
    assert orc.k_from_rate(576, 25, 100) == 144
    assert orc.k_from_rate(7, 0, 1) == 0 and orc.k_from_rate(7, 1, 1) == 7


def test_eq13_reproduces_printed_tflops():
    for c in GOLD["prefill_tflops"]["cases"]:
        f = orc.prefill_flops_model(c["layers"], c["dense_layers"], c["n_full"], c["n_kept"], c["width"])
        assert round(f / 1e12, 1) == c["printed"], c["model"]
    # the single-layer formula itself, by hand: 32*1*2*3^2 + 4*1*2^2*3
    assert orc.prefill_flops(1, 2, 3) == 32 * 2 * 9 + 4 * 4 * 3
