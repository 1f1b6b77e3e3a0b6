"""The checker's own rule for decisions that floating point takes (CPU only): a GPU decision may differ from the
fp64 oracle's only where the oracle's margin is below 1e-3; such flips are reported, anything else fails.
The "GPU" decisions here are made on the host in fp32, the precision the kernels decide in."""
import numpy as np
import pytest

from oracle import dl_oracle as orc
from tests import path_check as pc


def _fp32_selection(s64, k):
    """What a correct fp32 implementation selects: the oracle's rule applied to the fp32-rounded scores."""
    return orc.topk_select(s64.astype(np.float32).astype(np.float64), k)[1]


def test_selection_flip_inside_margin_is_reported_not_failed():
    # scores 3 and 7 differ by 1e-9: equal in fp32, so fp32 keeps the lower index, fp64 the larger score
    s = np.array([0.9, 0.1, 0.2, 0.5, 0.05, 0.0, -1.0, 0.5 + 1e-9, 0.3], dtype=np.float64)
    k = 2
    keep32 = _fp32_selection(s, k)
    keep64 = orc.topk_select(s, k)[1]
    assert keep32[3] == 1 and keep32[7] == 0 and keep64[7] == 1 and keep64[3] == 0
    flips = pc.selection_flips(s, keep32, k)
    assert sorted(i for i, _, _ in flips) == [3, 7] and all(ok for _, _, ok in flips)
    pc.assert_flips_in_margin(flips, "selection")            # tolerated


def test_selection_flip_outside_margin_fails():
    s = np.array([0.9, 0.1, 0.2, 0.5, 0.05, 0.0, -1.0, 0.6, 0.3], dtype=np.float64)
    wrong = orc.topk_select(s, 2)[1].copy()
    wrong[7], wrong[3] = 0, 1                                  # planted: 0.5 kept instead of 0.6 (gap 0.1)
    flips = pc.selection_flips(s, wrong, 2)
    assert len(flips) == 2
    with pytest.raises(AssertionError):
        pc.assert_flips_in_margin(flips, "selection")


def test_keep_flip_inside_margin_is_reported_not_failed():
    z = np.array([0.7, 1e-50, -0.2, -1e-50, 5e-4], dtype=np.float64)    # 1e-50 is +0 in fp32: dropped there
    m32 = orc.decode_keep(z.astype(np.float32).astype(np.float64))
    assert list(m32) == [1, 0, 0, 0, 1] and list(orc.decode_keep(z)) == [1, 1, 0, 0, 1]
    flips = pc.keep_flips(z, m32)
    assert [(b, ok) for b, _, ok in flips] == [(1, True)]
    pc.assert_flips_in_margin(flips, "keep")


def test_keep_flip_outside_margin_fails():
    z = np.array([0.7, 0.02, -0.2], dtype=np.float64)
    wrong = np.array([1, 0, 0], dtype=np.uint8)                # planted: logit 0.02 dropped
    flips = pc.keep_flips(z, wrong)
    assert [(b, ok) for b, _, ok in flips] == [(1, False)]
    with pytest.raises(AssertionError):
        pc.assert_flips_in_margin(flips, "keep")
