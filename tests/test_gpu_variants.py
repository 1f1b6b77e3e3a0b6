"""The paper's other operating points on the same kernels, chained GPU-vs-oracle parity at reduced batch and
depth: vision keep rates of 20 / 50 / 80 % and generated-token keep rates of 20 / 80 % (the ablation over
r^I and r^OT, Tab. 5), and a projector that hands over 144 vision tokens of which 57 are kept (the
TokenPacker setting of Sec. 4.2)."""
import pytest

from tests import path_check as pc

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("k_vis", [115, 288, 461])          # 20 / 50 / 80 % of 576
def test_vision_keep_rates(k_vis):
    rep = pc.run_chained(3, n_decode=4, B=2, L=1, shape={"k_vis": k_vis}, verbose=True)
    assert rep["score_maxabs"] <= pc.LOGIT_TOL


@pytest.mark.parametrize("rate", [0.2, 0.8])
def test_generated_keep_rates(rate):
    rep = pc.run_chained(2, n_decode=48, txt_keep_rate=rate, verbose=True)
    kept, total = (int(x) for x in rep["decode_kept"].split("/"))
    assert abs(kept - rate * total) <= 3                      # the bias was set on these very rows


def test_compressed_projector_144_to_57():
    pc.run_chained(3, n_decode=4, B=2, L=1, shape={"n_vis": 144, "k_vis": 57}, verbose=True)


def test_keep_every_vision_token_equals_dense_prefill():
    # r^I = 100 %: selection keeps everything and the path is dense causal attention on the full context
    pc.run_chained(2, n_decode=2, shape={"k_vis": 576}, verbose=True)
