"""Pins for the oracle's top-k selection (Eq. 11) and decode keep decision (Eq. 5 / 6)."""
import itertools

import numpy as np
import pytest

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl


def brute_topk(s, k):
    s = [(-np.inf if (x != x) else float(x)) for x in s]
    order = sorted(range(len(s)), key=lambda i: (-s[i], i))
    return sorted(order[:k])


def test_matches_brute_force_sort_on_tiny_inputs():
    rng = np.random.default_rng(0)
    for n in range(0, 9):
        for trial in range(20):
            # few distinct values => many ties
            s = rng.integers(-2, 3, size=n).astype(np.float32)
            for k in range(n + 1):
                idx, keep = orc.topk_select(s, k)
                assert list(idx) == brute_topk(s, k)
                assert keep.sum() == k and len(idx) == k
                assert all(keep[i] == 1 for i in idx)


def test_all_orderings_of_distinct_values():
    vals = [0.5, -1.0, 3.0, 2.0, -0.25]
    for perm in itertools.permutations(vals):
        for k in range(6):
            idx, _ = orc.topk_select(np.array(perm), k)
            top = sorted(vals, reverse=True)[:k]
            assert sorted(perm[i] for i in idx) == sorted(top)
            assert list(idx) == sorted(idx)


def test_order_property_and_ascending_output():
    rng = np.random.default_rng(5)
    s = np.round(rng.normal(size=300), 1)
    for k in (0, 1, 75, 299, 300):
        idx, keep = orc.topk_select(s, k)
        assert np.all(np.diff(idx) > 0)
        kept, dropped = np.flatnonzero(keep == 1), np.flatnonzero(keep == 0)
        for i in kept:
            for j in dropped:
                assert s[i] > s[j] or (s[i] == s[j] and i < j)


def test_degenerate_cases():
    idx, keep = orc.topk_select(np.ones(10), 4)           # all equal: lowest indices win
    assert list(idx) == [0, 1, 2, 3]
    idx, _ = orc.topk_select(np.array([0.0, -0.0, 0.0, -0.0]), 2)   # -0 == +0: a tie
    assert list(idx) == [0, 1]
    idx, _ = orc.topk_select(np.array([-0.0, 0.0, -1.0]), 1)
    assert list(idx) == [0]
    idx, _ = orc.topk_select(np.array([np.nan, -np.inf, 1.0, np.nan]), 3)   # NaN ranks as -inf
    assert list(idx) == [0, 1, 2]
    idx, _ = orc.topk_select(np.array([np.inf, 1.0, np.inf]), 2)
    assert list(idx) == [0, 2]
    assert orc.topk_select(np.arange(5.0), 0)[1].sum() == 0
    assert orc.topk_select(np.arange(5.0), 5)[1].sum() == 5
    with pytest.raises(ValueError):
        orc.topk_select(np.arange(5.0), 6)


def test_batch_form_respects_ragged_lengths():
    rng = np.random.default_rng(6)
    score = rng.normal(size=(3, 12)).astype(np.float32)
    score[1, 8:] = 100.0           # padding slots with huge scores must never be selected
    n_vis, k = np.array([12, 8, 5]), np.array([3, 8, 0])
    kept_idx, keep = orc.prefill_select(score, n_vis, k)
    assert kept_idx.shape == (3, 8)
    assert list(kept_idx[0, :3]) == brute_topk(score[0], 3) and np.all(kept_idx[0, 3:] == -1)
    assert list(kept_idx[1]) == list(range(8)) and keep[1, 8:].sum() == 0
    assert np.all(kept_idx[2] == -1) and keep[2].sum() == 0
    assert list(keep.sum(axis=1)) == [3, 8, 0]


def test_decode_keep_counts_positive_logits():
    z = np.array([0.3, -0.1, 0.0, -0.0, 1e-30, -1e-30, np.nan, np.inf, -np.inf])
    m = orc.decode_keep(z)
    assert list(m) == [1, 0, 0, 0, 1, 0, 0, 1, 0]          # strict '>' ; NaN drops
    assert m.sum() == sum(1 for v in z if v > 0)
    assert list(orc.decode_keep(np.array([0.5, 1.5]), threshold=1.0)) == [0, 1]
    # alternating-sign logits reproduce the paper's "Structure" static mask (every other token)
    alt = np.where(np.arange(10) % 2 == 0, 1.0, -1.0)
    assert list(orc.decode_keep(alt)) == list(wl.static_keep_pattern("structure", 10))


def test_nocache_mask_keeps_the_last_generated_token():
    """Eq. 12 / text above Eq. 6: all generated tokens are decided at once and the last one is kept."""
    z = np.array([[0.5, -1.0, 0.0, -2.0, 9.0], [-1.0, -1.0, -1.0, -1.0, -1.0], [3.0, 3.0, 3.0, 3.0, 3.0]])
    m = orc.nocache_keep(z, np.array([4, 5, 0]))
    assert m.tolist() == [[1, 0, 0, 1, 0], [0, 0, 0, 0, 1], [0, 0, 0, 0, 0]]
    # brute force over random inputs: positives, plus the last valid slot, nothing in the padding
    rng = np.random.default_rng(9)
    z = rng.normal(size=(6, 17))
    n = rng.integers(0, 18, size=6)
    m = orc.nocache_keep(z, n)
    for b in range(6):
        for i in range(17):
            want = i < n[b] and (z[b, i] > 0 or i == n[b] - 1)
            assert m[b, i] == int(want)
    # without the forced token it is Eq. 6's per-token decision
    assert np.array_equal(orc.nocache_keep(z, None)[:, :-1], orc.decode_keep(z)[:, :-1])


def test_prefill_keep_mask_ragged_batch_by_brute_force():
    """M = M^I u {1}^{N_T} (Sec. 3.3.3) for a batch whose sequences have different numbers of vision AND text
    tokens: written out slot by slot (no slicing), and applied through append_rows it must leave exactly
    k_b + N_T(b) rows, the kept vision rows first and in order, then the text rows."""
    rng = np.random.default_rng(5)
    B, nv_max = 4, 9
    n_vis = np.array([9, 4, 0, 7])
    n_text = np.array([3, 5, 2, 0])
    k = np.array([2, 4, 0, 3])
    score = rng.normal(size=(B, nv_max))
    _, keep_vis = orc.prefill_select(score, n_vis, k)
    m = orc.prefill_keep_mask(keep_vis, n_vis, n_text)
    assert m.shape == (B, nv_max + 5)
    for b in range(B):
        for t in range(m.shape[1]):
            if t < nv_max:
                want = 1 if (t < n_vis[b] and keep_vis[b, t]) else 0
            else:
                want = 1 if t - nv_max < n_text[b] else 0
            assert m[b, t] == want, (b, t)
        assert m[b].sum() == k[b] + n_text[b]
    # through the compaction: source rows are numbered, so the cache shows which rows arrived and in what order
    T = m.shape[1]
    src = np.arange(B * T, dtype=np.float32).reshape(B, T, 1, 1)
    cache = np.full((B, 1, T, 1), -1.0, np.float32)
    ln = np.zeros(B, np.int32)
    st, cnt = orc.append_rows(src, src, m, None, cache, cache.copy(), ln)
    assert st == orc.OK and list(ln) == list(k + n_text)
    for b in range(B):
        rows = [t for t in range(nv_max) if t < n_vis[b] and keep_vis[b, t]] + [nv_max + j for j in range(n_text[b])]
        assert list(cache[b, 0, : ln[b], 0]) == [float(b * T + t) for t in rows]
