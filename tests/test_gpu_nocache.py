"""Decoding WITHOUT KV cache (Eq. 12): all generated tokens are decided at once (last one kept), the
reduced set S^{P*} u S^{OT*} is rebuilt by compaction and attended causally.  The GPU result is
compared with the definition itself: masked attention over the FULL, uncompacted context (Eq. 7
with diag(G) = 1), restricted to the rows that are computed."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl
from tests import path_check as pc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype,H,D", [("bf16", 4, 128), ("f32", 2, 64)])
def test_decode_without_cache_step(dtype, H, D):
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[2].scaled(B=2, hidden=512, pred_hidden=128, n_heads=H, head_dim=D, dtype=dtype)
    B, nv, nt, ng = 2, 40, 10, 30
    n_gen = np.array([ng, 17], np.int32)
    cap = 128
    rng = np.random.default_rng(11)
    p = wl.make_predictor(cfg, "txt", b2=0.0)
    x_gen = wl.host_normal(cfg, wl.S_X_TXT, (B, ng, cfg.hidden))
    keep_vis = (rng.random((B, nv)) < 0.3).astype(np.uint8)
    pre = [wl.host_normal(cfg, s, (B, nv + nt, H, D)) for s in (wl.S_Q, wl.S_K, wl.S_V)]          # q, k, v
    gen = [wl.host_normal(cfg, s, (B, ng, H, D)) for s in (wl.S_DEC_Q, wl.S_DEC_K, wl.S_DEC_V)]
    tdt = wl.torch_dtype(dtype)
    D_ = lambda a: wl.to_torch(a, dtype, DEV)
    ctx = dl.Context(cfg.hidden, H, D, cfg.pred_hidden, tdt, 0, max_batch=B, max_rows=B * ng, cap=cap)
    pd = dl.Predictor(D_(p.w1), torch.from_numpy(p.b1).to(DEV), torch.from_numpy(p.w2).to(DEV), p.b2)

    # ---- Eq. 12: decisions for all generated tokens, last one forced
    logit = torch.zeros(B, ng, dtype=torch.float32, device=DEV)
    keep_gen = torch.full((B, ng), 7, dtype=torch.uint8, device=DEV)
    n_gen_d = torch.from_numpy(n_gen).to(DEV)
    ctx.decode_nocache_select(pd, D_(x_gen), n_gen_d, logit, keep_gen)
    z, m = logit.cpu().numpy(), keep_gen.cpu().numpy()
    z_ref = orc.predictor_logits(x_gen, p.w1, p.b1, p.w2, p.b2)
    for b in range(B):
        assert np.abs(z[b, : n_gen[b]] - z_ref[b, : n_gen[b]]).max() <= pc.LOGIT_TOL
    assert np.array_equal(m, orc.nocache_keep(z.astype(np.float64), n_gen))           # bit-exact on its own logits
    m_ref = orc.nocache_keep(z_ref, n_gen)
    for b, i in np.argwhere(m != m_ref):
        assert abs(z_ref[b, i]) < pc.MARGIN
    assert all(m[b, n_gen[b] - 1] == 1 for b in range(B)) and not m[1, n_gen[1]:].any()

    # ---- reduced set: kept vision rows, all text rows, kept generated rows, in order
    i32 = dict(dtype=torch.int32, device=DEV)
    caches = [torch.zeros(B, H, cap, D, dtype=tdt, device=DEV) for _ in range(3)]                # q, k, v
    ln = torch.zeros(B, **i32)
    lq = torch.zeros(B, **i32)
    kv_d = torch.from_numpy(keep_vis).to(DEV)
    t_pre = torch.full((B,), nv + nt, **i32)
    ctx.compact_kv(D_(pre[0]), None, kv_d, t_pre, caches[0], None, lq, commit=True)
    ctx.compact_kv(D_(pre[1]), D_(pre[2]), kv_d, t_pre, caches[1], caches[2], ln, commit=True)
    ctx.compact_kv(D_(gen[0]), None, keep_gen, n_gen_d, caches[0], None, lq, commit=True)
    ctx.compact_kv(D_(gen[1]), D_(gen[2]), keep_gen, n_gen_d, caches[1], caches[2], ln, commit=True)
    lens = ln.cpu().numpy()
    want_len = keep_vis.sum(axis=1) + nt + m.sum(axis=1)
    assert np.array_equal(lens, want_len) and np.array_equal(lq.cpu().numpy(), want_len)

    # ---- attention over the reduced set vs the masked definition on the full context
    n_max = int(lens.max())
    out = torch.zeros(B, n_max, H, D, dtype=tdt, device=DEV)
    scale = 1 / np.sqrt(D)
    ctx.sparse_attn_prefill(caches[0], caches[1], caches[2], ln, n_max, scale, out)
    got = wl.from_torch(out)
    for b in range(B):
        full_mask = np.concatenate([keep_vis[b], np.ones(nt, np.uint8), m[b, : n_gen[b]]])
        rows = np.flatnonzero(full_mask)
        for h in range(H):
            q, k, v = (np.concatenate([pre[j][b, :, h], gen[j][b, : n_gen[b], h]]) for j in range(3))
            ref = orc.attention_masked_full(q, k, v, full_mask, scale)[rows]
            pc.check_att(got[b, : lens[b], h], ref, f"no-cache attention b={b} h={h}")
            # the cache itself is the ordered gather of the kept rows
            assert np.array_equal(pc.dev_bits(caches[1][b, h, : lens[b]]), pc.host_bits(k[rows], dtype))
    assert ctx.device_status()[0] == 0
