"""The paper's own predictors on the GPU against their CPU oracle (App. "Details of Predictor Architecture";
Eq. 5 argmax, Eq. 11 ranking by the second decision value): decision values within the logit tolerance, the
selection equal to the oracle's selection of the GPU's own scores (bit-exact) and within the margin of the
oracle's own, the argmax decision equal to the comparison of the GPU's own two values.  The margin inside which a
decision may differ from the oracle's is twice the logit tolerance here (path_check.MARGIN_CHAIN): the chain's
activations are rounded to bf16 between its ten layers, so its values meet the logit tolerance and no more."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from oracle import predictor_paper as pp
from paper_2412_00876_b200 import workloads as wl
from tests import path_check as pc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _to_dev(params):
    """make_predictor_paper's dictionary on the device: matrices bf16, vectors float32 (w3 stays float32)."""
    def conv(k, v):
        if isinstance(v, dict):
            return {kk: conv(kk, vv) for kk, vv in v.items()}
        if isinstance(v, list):
            return [conv(k, x) for x in v]
        if v.ndim == 2 and k != "w3":
            return wl.to_torch(v, "bf16", DEV)
        return torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to(DEV)
    return conv("", params)


def _ctx(cfg, B, rows):
    from paper_2412_00876_b200 import binding as dl
    return dl.Context(cfg.hidden, cfg.n_heads, cfg.head_dim, cfg.pred_hidden, torch.bfloat16, 0, max_batch=B,
                      max_rows=rows, cap=64)


@pytest.mark.parametrize("cid,B,n_max,n_vis,k", [(2, 2, 576, [576, 431], [144, 100]),
                                                 (5, 1, 2880, [2880], [576]),
                                                 (2, 3, 100, [100, 1, 64], [20, 1, 0])])
def test_image_predictor_and_selection(cid, B, n_max, n_vis, k):
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[cid]
    params = wl.make_predictor_paper(cfg, "img")
    x = wl.host_normal(cfg, wl.S_X_VIS, (B, n_max, cfg.hidden))
    xd = wl.to_torch(x, "bf16", DEV)
    for b in range(B):
        xd[b, n_vis[b]:] = float("nan")                       # padding rows are unspecified: make them hostile
    ctx = _ctx(cfg, B, B * n_max)
    p = dl.Predictor2(_to_dev(params))
    scratch = ctx.predictor2_scratch(B * n_max)
    i32 = dict(dtype=torch.int32, device=DEV)
    d_out = torch.empty(B * n_max, 2, dtype=torch.float32, device=DEV)
    score = torch.empty(B, n_max, dtype=torch.float32, device=DEV)
    k_max = max(1, max(k))
    kept = torch.empty(B, k_max, **i32)
    keep = torch.empty(B, n_max, dtype=torch.uint8, device=DEV)
    nv, kd = torch.tensor(n_vis, **i32), torch.tensor(k, **i32)
    ctx.prefill_select2(p, xd, nv, kd, scratch, d_out, score, kept, keep)
    D_gpu = d_out.cpu().numpy().reshape(B, n_max, 2).astype(np.float64)
    D_ref = pp.image_predictor(x, params, n_vis)
    err = max(np.abs(D_gpu[b, : n_vis[b]] - D_ref[b, : n_vis[b]]).max() for b in range(B) if n_vis[b])
    assert err <= pc.LOGIT_TOL, err
    for b in range(B):
        assert np.all(D_gpu[b, n_vis[b]:] == 0)               # padding rows
    s_gpu = score.cpu().numpy().astype(np.float64)
    assert all(np.array_equal(s_gpu[b, : n_vis[b]], D_gpu[b, : n_vis[b], 1]) for b in range(B))   # the score IS D[:,2]
    # stage-isolated: the selection is the oracle's selection of the GPU's own scores
    idx_iso, keep_iso = orc.prefill_select(s_gpu, n_vis, np.array(k), k_max)
    assert np.array_equal(keep.cpu().numpy(), keep_iso) and np.array_equal(kept.cpu().numpy(), idx_iso)
    # chained: against the oracle's own scores only inside the margin
    for b in range(B):
        fl = pc.selection_flips(pp.ranking_score(D_ref[b, : n_vis[b]]), keep.cpu().numpy()[b, : n_vis[b]], k[b],
                                margin=pc.MARGIN_CHAIN)
        pc.assert_flips_in_margin(fl, f"selection by D[:,2] (sequence {b})")
    # the argmax decision of Eq. 5 on the same values
    km = torch.empty(B, n_max, dtype=torch.uint8, device=DEV)
    ctx.predictor2_values(p, xd, nv, scratch, d_out=d_out, keep_out=km)
    D2 = d_out.cpu().numpy().reshape(B, n_max, 2)
    assert np.array_equal(km.cpu().numpy(), (D2[..., 1] > D2[..., 0]).astype(np.uint8))
    for b in range(B):
        m_ref = pp.decision_keep(D_ref[b, : n_vis[b]])
        for i in np.flatnonzero(m_ref != km.cpu().numpy()[b, : n_vis[b]]):
            assert abs(D_ref[b, i, 1] - D_ref[b, i, 0]) < pc.MARGIN_CHAIN
    assert ctx.device_status()[0] == 0
    ctx.close()


@pytest.mark.parametrize("cid,B", [(2, 1), (4, 64), (5, 16)])
def test_text_predictor_decode_decision(cid, B):
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[cid]
    params = wl.make_predictor_paper(cfg, "txt")
    x = wl.host_normal(cfg, wl.S_X_TXT, (B, cfg.hidden))
    ctx = _ctx(cfg, B, B)
    p = dl.Predictor2(_to_dev(params))
    scratch = ctx.predictor2_scratch(B)
    d_out = torch.empty(B, 2, dtype=torch.float32, device=DEV)
    keep = torch.empty(B, dtype=torch.uint8, device=DEV)
    ctx.decode_keep2(p, wl.to_torch(x, "bf16", DEV), scratch, d_out, keep)
    D_gpu = d_out.cpu().numpy().astype(np.float64)
    D_ref = pp.text_predictor(x, params)
    assert np.abs(D_gpu - D_ref).max() <= pc.LOGIT_TOL
    assert np.array_equal(keep.cpu().numpy(), (D_gpu[:, 1] > D_gpu[:, 0]).astype(np.uint8))
    for b in np.flatnonzero(pp.decision_keep(D_ref) != keep.cpu().numpy()):
        assert abs(D_ref[b, 1] - D_ref[b, 0]) < pc.MARGIN_CHAIN
    if B >= 16:
        assert 0 < keep.sum().item() < B                     # decisions of both kinds
    assert ctx.device_status()[0] == 0
    ctx.close()
