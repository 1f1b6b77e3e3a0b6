"""Chained GPU-vs-oracle parity: the whole path (select -> compaction -> prefill attention ->
decode steps with keep decision, attention and append), every stage checked, flips logged."""
import pytest

from tests import path_check as pc

pytestmark = pytest.mark.gpu


def test_config1_toy_fp32_full():
    rep = pc.run_chained(1, verbose=True)
    assert rep["score_maxabs"] < 1e-4


def test_config2_7b_single_layer_full():
    rep = pc.run_chained(2, verbose=True)          # 576 -> 144 vision tokens, 64 prompt, 256 decode steps
    assert rep["decode_kept"].split("/")[1] == "256"


@pytest.mark.parametrize("cid", [3, 4, 5])
def test_batched_configs_scaled(cid):
    # the batched configurations at their own widths, with 2 sequences, 2 layers and 12 decode steps
    pc.run_chained(cid, n_decode=12, B=2, L=2, verbose=True)


def test_ragged_batch():
    pc.run_chained(3, n_decode=6, B=3, L=1, ragged=True, verbose=True)
