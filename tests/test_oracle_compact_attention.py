"""Pins for the oracle's compaction (Eq. 5 set builder, Eq. 6 append) and attention
(Eq. 7 with diag(G)=1; Eq. 1 / Eq. 6 on the reduced set)."""
import json
import os

import numpy as np

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


# ------------------------------------------------------------------ compaction
def _src(B, T, H, D, seed=0):
    rng = np.random.default_rng(seed)
    k = rng.integers(0, 2 ** 16, size=(B, T, H, D), dtype=np.uint16)
    v = rng.integers(0, 2 ** 16, size=(B, T, H, D), dtype=np.uint16)
    return k, v


def test_compaction_is_a_bitwise_ordered_gather():
    B, T, H, D, cap = 2, 11, 3, 4, 16
    k, v = _src(B, T, H, D)
    keep = np.array([[1, 0, 0, 1, 1, 0, 1, 0, 0, 0, 1], [0] * 10 + [1]], dtype=np.uint8)
    kc, vc = np.zeros((B, H, cap, D), np.uint16), np.zeros((B, H, cap, D), np.uint16)
    ln = np.zeros(B, dtype=np.int32)
    st, cnt = orc.append_rows(k, v, keep, None, kc, vc, ln)
    assert st == orc.OK and list(ln) == [5, 1] and list(cnt) == [5, 1]
    for b in range(B):
        kept = np.flatnonzero(keep[b])
        for j, t in enumerate(kept):
            for h in range(H):
                assert np.array_equal(kc[b, h, j], k[b, t, h]) and np.array_equal(vc[b, h, j], v[b, t, h])
        assert not kc[b, :, len(kept):].any()       # nothing written past the new length


def test_length_accounting_matches_paper_totals():
    g = GOLD["total_tokens_computed"]
    kv = g["image_kept"]
    for c in g["cases"]:
        n_img, H, D = 576, 1, 2
        T = n_img + c["text"]
        k, v = _src(1, T, H, D, seed=c["text"])
        score = np.random.default_rng(c["total"]).normal(size=(1, n_img))
        _, keep_vis = orc.prefill_select(score, None, np.array([kv]))
        mask = orc.prefill_keep_mask(keep_vis, None, np.array([c["text"]]))
        cap = 1024
        kc, vc = np.zeros((1, H, cap, D), np.uint16), np.zeros((1, H, cap, D), np.uint16)
        ln = np.zeros(1, dtype=np.int32)
        orc.append_rows(k, v, mask, None, kc, vc, ln)
        assert ln[0] == kv + c["text"]
        # decode: every generated token kept -> the paper's total
        for t in range(c["output"]):
            ks, vs = _src(1, 1, H, D, seed=100 + t)
            orc.append_rows(ks, vs, np.ones((1, 1), np.uint8), None, kc, vc, ln)
        assert ln[0] == c["total"]


def test_keep_all_is_a_transposed_copy_and_idempotent():
    B, T, H, D = 2, 7, 3, 4
    k, v = _src(B, T, H, D, 3)
    kc, vc = np.zeros((B, H, T, D), np.uint16), np.zeros((B, H, T, D), np.uint16)
    ln = np.zeros(B, dtype=np.int32)
    orc.append_rows(k, v, None, None, kc, vc, ln)
    assert np.array_equal(kc, k.transpose(0, 2, 1, 3)) and np.array_equal(vc, v.transpose(0, 2, 1, 3))
    # compacting the compact cache again with keep-all changes nothing
    kc2, vc2 = np.zeros_like(kc), np.zeros_like(vc)
    ln2 = np.zeros(B, dtype=np.int32)
    orc.append_rows(kc.transpose(0, 2, 1, 3), vc.transpose(0, 2, 1, 3), None, ln, kc2, vc2, ln2)
    assert np.array_equal(kc2, kc) and np.array_equal(vc2, vc) and np.array_equal(ln2, ln)


def test_ragged_sources_append_and_capacity():
    B, T, H, D, cap = 3, 6, 2, 2, 8
    k, v = _src(B, T, H, D, 4)
    kc, vc = np.zeros((B, H, cap, D), np.uint16), np.zeros((B, H, cap, D), np.uint16)
    ln = np.array([0, 5, 7], dtype=np.int32)
    keep = np.ones((B, T), np.uint8)
    before = kc.copy()
    st, cnt = orc.append_rows(k, v, keep, np.array([6, 3, 2]), kc, vc, ln)
    assert st == orc.ERR_CAPACITY                      # sequence 2: 7 + 2 > 8 -> untouched
    assert list(ln) == [6, 8, 7] and list(cnt) == [6, 3, 0]
    assert np.array_equal(kc[2], before[2])
    assert np.array_equal(kc[1, :, 5:8], k[1, :3].transpose(1, 0, 2))
    # commit=False writes the rows but leaves the lengths alone (several layers share one length)
    ln3 = np.array([1, 1, 1], dtype=np.int32)
    orc.append_rows(k, v, keep, np.array([1, 1, 1]), kc, vc, ln3, commit=False)
    assert list(ln3) == [1, 1, 1] and np.array_equal(kc[0, :, 1], k[0, 0])


# ------------------------------------------------------------------ attention
def dense_causal_textbook(q, k, v, scale):
    """softmax(Q K^T * scale + causal) V with an additive -inf mask, written with matrices."""
    n = q.shape[0]
    z = (q @ k.T) * scale + np.triu(np.full((n, n), -np.inf), 1)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    return (p / p.sum(axis=1, keepdims=True)) @ v


def _qkv(n, d, seed):
    rng = np.random.default_rng(seed)
    return rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=(n, d))


def test_keep_everything_equals_dense_causal_attention():
    q, k, v = _qkv(37, 16, 0)
    ref = dense_causal_textbook(q, k, v, 0.25)
    assert np.allclose(orc.attention_masked_full(q, k, v, np.ones(37), 0.25), ref, atol=1e-13)
    assert np.allclose(orc.attention_prefill_compact(q, k, v, 37, 0.25), ref, atol=1e-13)
    # decode form, token by token, against the same dense result
    for i in (0, 1, 17, 36):
        o = orc.attention_decode_compact(q[i], k[i], v[i], k, v, i, 0.25)
        assert np.allclose(o, ref[i], atol=1e-13)


def test_compact_cache_equals_full_context_with_dropped_tokens_masked():
    n, d, scale = 48, 8, 1 / np.sqrt(8)
    q, k, v = _qkv(n, d, 1)
    mask = wl.static_keep_pattern("random", n).copy()
    mask[-1] = 0                                   # last token dropped too
    full = orc.attention_masked_full(q, k, v, mask, scale)
    kept = np.flatnonzero(mask)
    # prefill form: the kept rows, compacted, attend causally among themselves
    comp = orc.attention_prefill_compact(q[kept], k[kept], v[kept], len(kept), scale)
    assert np.allclose(comp, full[kept], atol=1e-13)
    # decode form: token i sees the kept tokens before it plus itself, kept or not
    for i in range(n):
        prev = kept[kept < i]
        o = orc.attention_decode_compact(q[i], k[i], v[i], k[prev], v[prev], len(prev), scale)
        assert np.allclose(o, full[i], atol=1e-13), i
    # and the -inf form of the textbook routine agrees with the masked definition
    z = (q @ k.T) * scale
    vis = np.tril(np.ones((n, n), bool)) & (mask.astype(bool)[None, :] | np.eye(n, dtype=bool))
    z = np.where(vis, z, -np.inf)
    p = np.exp(z - z.max(axis=1, keepdims=True))
    assert np.allclose((p / p.sum(axis=1, keepdims=True)) @ v, full, atol=1e-13)


def test_closed_forms():
    n, d = 9, 5
    q, k, v = _qkv(n, d, 2)
    # zero queries: uniform weights -> running mean of the visible values
    o = orc.attention_prefill_compact(np.zeros((n, d)), k, v, n, 0.7)
    assert np.allclose(o, np.cumsum(v, axis=0) / np.arange(1, n + 1)[:, None], atol=1e-14)
    o = orc.attention_decode_compact(np.zeros(d), k[0], v[0], k[1:], v[1:], n - 1, 0.7)
    assert np.allclose(o, v.mean(axis=0), atol=1e-14)
    # a single visible row returns its value; empty cache -> the current token's value
    assert np.allclose(orc.attention_prefill_compact(q, k, v, n, 1.0)[0], v[0])
    assert np.allclose(orc.attention_decode_compact(q[0], k[0], v[3], k, v, 0, 1.0), v[3])
    # equal values -> that value; outputs are convex combinations of the values
    same = np.tile(v[:1], (n, 1))
    assert np.allclose(orc.attention_prefill_compact(q, k, same, n, 1.0), same, atol=1e-14)
    o = orc.attention_prefill_compact(q, k, v, n, 1.0)
    for i in range(n):
        assert np.all(o[i] <= v[: i + 1].max(axis=0) + 1e-14) and np.all(o[i] >= v[: i + 1].min(axis=0) - 1e-14)
    # two rows, by hand: weights are sigmoid of the score difference
    z0, z1 = q[1] @ k[0], q[1] @ k[1]
    w1 = 1 / (1 + np.exp(z0 - z1))
    assert np.allclose(o[1], (1 - w1) * v[0] + w1 * v[1], atol=1e-14)
    # scale enters as a multiplier of q.k
    a = orc.attention_decode_compact(q[0], k[0], v[0], k, v, n, 0.5)
    b = orc.attention_decode_compact(0.5 * q[0], k[0], v[0], k, v, n, 1.0)
    assert np.allclose(a, b, atol=1e-14)


def test_shift_and_permutation_invariance_in_decode():
    n, d = 20, 6
    q, k, v = _qkv(n, d, 3)
    base = orc.attention_decode_compact(q[0], k[0], v[0], k[1:], v[1:], n - 1, 0.3)
    # adding c*q/|q|^2 to every key shifts every score by the same constant
    shift = 5.0 * q[0] / (q[0] @ q[0])
    o = orc.attention_decode_compact(q[0], k[0] + shift, v[0], k[1:] + shift, v[1:], n - 1, 0.3)
    assert np.allclose(o, base, atol=1e-12)
    perm = np.random.default_rng(0).permutation(n - 1)
    o = orc.attention_decode_compact(q[0], k[0], v[0], k[1:][perm], v[1:][perm], n - 1, 0.3)
    assert np.allclose(o, base, atol=1e-13)
    # rows past the valid length are never read
    kk, vv = k[1:].copy(), v[1:].copy()
    kk[10:], vv[10:] = np.nan, np.nan
    o = orc.attention_decode_compact(q[0], k[0], v[0], kk, vv, 10, 0.3)
    assert np.all(np.isfinite(o))


def test_dropped_token_contributes_only_to_its_own_step():
    """Sec. 3.3.2: the current token always takes part in its own attention, even when its
    K/V are not kept; afterwards it is gone."""
    n, d, scale = 12, 4, 0.5
    q, k, v = _qkv(n, d, 4)
    mask = np.ones(n, dtype=np.uint8)
    mask[5] = 0
    base = orc.attention_masked_full(q, k, v, mask, scale)
    v2 = v.copy()
    v2[5] += 10.0
    pert = orc.attention_masked_full(q, k, v2, mask, scale)
    changed = np.flatnonzero(np.abs(pert - base).max(axis=1) > 1e-12)
    assert list(changed) == [5]
    mask[5] = 1                                       # kept instead: every later row changes
    base = orc.attention_masked_full(q, k, v, mask, scale)
    pert = orc.attention_masked_full(q, k, v2, mask, scale)
    assert list(np.flatnonzero(np.abs(pert - base).max(axis=1) > 1e-12)) == list(range(5, n))


def test_planted_mistakes_are_caught():
    """The pins above must fail for plausible mistakes; check two of them explicitly."""
    n, d = 10, 4
    q, k, v = _qkv(n, d, 5)
    ref = dense_causal_textbook(q, k, v, 0.5)
    # (1) forgetting the current token in decode
    wrong = orc.attention_decode_compact(q[4], k[3], v[3], k, v, 3, 0.5)
    assert not np.allclose(wrong, ref[4], atol=1e-6)
    # (2) a non-strict causal boundary (one extra future row)
    wrong = orc.attention_decode_compact(q[4], k[5], v[5], k, v, 5, 0.5)
    assert not np.allclose(wrong, ref[4], atol=1e-6)
