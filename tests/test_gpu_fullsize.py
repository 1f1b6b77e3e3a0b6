"""Parity at full workload size, in the launch configuration the benchmark times.

The batched configurations are too large for the oracle to recompute whole, so the path is run
once at full size (same BatchRunner as bench.py) and sampled outputs are recomputed one by one:
predictor rows, whole-sequence selections, compacted cache slices, prefill attention rows and
decode attention outputs of sampled (layer, sequence, head) triples, plus properties that hold
at any size (kept counts, lengths, untouched rows)."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl
from tests import path_check as pc

pytestmark = pytest.mark.gpu


def _f64(t):
    return wl.from_torch(t)


@pytest.mark.parametrize("cid,n_steps", [(3, 24), (4, 8), (5, 8)])
def test_full_size_sampled(cid, n_steps):
    from paper_2412_00876_b200.runner import BatchRunner
    free, _ = torch.cuda.mem_get_info()
    cfg = wl.CONFIGS[cid]
    need = 2 * cfg.n_layers * cfg.B * cfg.n_heads * cfg.cap * cfg.head_dim * 2 * 1.4
    if free < need:
        pytest.skip("not enough free device memory for the full-size caches")
    r = BatchRunner(cfg, device=0)
    rng = np.random.default_rng(cid)
    B, L, H, D = cfg.B, cfg.n_layers, cfg.n_heads, cfg.head_dim
    scale = 1 / np.sqrt(D)
    r.prefill()
    torch.cuda.synchronize()

    # ---- a1: sampled predictor rows; a2: every sequence's selection from the GPU's own scores
    s_gpu = r.score.cpu().numpy()
    p = r.p_img_host
    for (b, i) in zip(rng.integers(0, B, 24), rng.integers(0, cfg.n_vis, 24)):
        ref = orc.predictor_logits(_f64(r.x_vis[b, i]), p.w1, p.b1, p.w2, p.b2)
        assert abs(s_gpu[b, i] - ref) <= pc.LOGIT_TOL
    keep = r.keep_vis.cpu().numpy()
    idx_ref, keep_ref = orc.prefill_select(s_gpu.astype(np.float64), None, np.full(B, cfg.k_vis), cfg.k_vis)
    assert np.array_equal(keep, keep_ref) and np.array_equal(r.kept_idx.cpu().numpy(), idx_ref)
    assert np.all(keep.sum(axis=1) == cfg.k_vis)
    lens0 = r.cache_len.cpu().numpy()
    assert np.all(lens0 == cfg.n0)

    # ---- a3: sampled cache slices equal the kept source rows, bit for bit
    kept_rows = [np.concatenate([np.flatnonzero(keep[b]), np.arange(cfg.n_vis, r.T)]) for b in range(B)]
    triples = [(int(rng.integers(0, L)), int(rng.integers(0, B)), int(rng.integers(0, H))) for _ in range(12)]
    triples += [(L - 1, B - 1, H - 1), (0, 0, 0)]
    for (l, b, h) in triples:
        src_k = r.k_src[l % r.src_pool][b, :, h].cpu()
        src_v = r.v_src[l % r.src_pool][b, :, h].cpu()
        rows = torch.from_numpy(kept_rows[b])
        assert torch.equal(r.k_cache[l][b, h, : cfg.n0].cpu().view(torch.int16), src_k[rows].view(torch.int16))
        assert torch.equal(r.v_cache[l][b, h, : cfg.n0].cpu().view(torch.int16), src_v[rows].view(torch.int16))

    # ---- a4: prefill attention of the last layer (the buffer the runner keeps), sampled (b, h), sampled rows
    l = L - 1
    out = r.prefill_out
    for (b, h) in [(0, 0), (B - 1, H - 1), (int(rng.integers(0, B)), int(rng.integers(0, H)))]:
        q = _f64(r.q_src[l % r.src_pool][b, :, h])[kept_rows[b]]
        k, v = _f64(r.k_cache[l][b, h, : cfg.n0]), _f64(r.v_cache[l][b, h, : cfg.n0])
        ref = orc.attention_prefill_compact(q, k, v, cfg.n0, scale)
        pc.check_att(_f64(out[b, :, h]), ref, f"prefill attention b={b} h={h}")

    # ---- a5-a7: decode steps; the last one is checked on sampled triples
    for t in range(n_steps - 1):
        r.decode_step(t)
    torch.cuda.synchronize()
    lens_before = r.cache_len.cpu().numpy().copy()
    t = n_steps - 1
    r.decode_step(t)
    torch.cuda.synchronize()
    i = t % r.step_pool
    z = r.logit.cpu().numpy()
    m = r.keep_t.cpu().numpy()
    pt = r.p_txt_host
    z_ref = orc.predictor_logits(_f64(r.x_dec[i]), pt.w1, pt.b1, pt.w2, pt.b2)
    assert np.abs(z - z_ref).max() <= pc.LOGIT_TOL
    assert np.array_equal(m, orc.decode_keep(z.astype(np.float64)))
    for b in np.flatnonzero(m != orc.decode_keep(z_ref)):
        assert abs(z_ref[b]) < pc.MARGIN
    lens_after = r.cache_len.cpu().numpy()
    assert np.array_equal(lens_after, lens_before + m)
    assert lens_before.min() >= cfg.n0 and lens_before.max() <= cfg.n0 + t
    for (l, b, h) in triples:
        n = int(lens_before[b])
        ref = orc.attention_decode_compact(_f64(r.q_dec[i, l, b, h]), _f64(r.k_dec[i, l, b, h]),
                                           _f64(r.v_dec[i, l, b, h]), _f64(r.k_cache[l][b, h, :n]),
                                           _f64(r.v_cache[l][b, h, :n]), n, scale)
        pc.check_att(_f64(r.dec_out[l, b, h]), ref, f"decode attention l={l} b={b} h={h}")
        if m[b]:
            assert torch.equal(r.k_cache[l][b, h, n].view(torch.int16), r.k_dec[i, l, b, h].view(torch.int16))
            assert torch.equal(r.v_cache[l][b, h, n].view(torch.int16), r.v_dec[i, l, b, h].view(torch.int16))
    code, detail = r.ctx.device_status()
    assert code == 0, (code, detail)
    r.close()
