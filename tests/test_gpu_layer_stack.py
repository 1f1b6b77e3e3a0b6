"""Decode over a layer stack whose decision is taken after the l-th layer (Sec. 3.3.1): the first l layers keep
every token, the remaining layers share the decision.  The whole stack runs through dl_decode_step_stack beside the
oracle, layer by layer; the token counts the two kinds of layers end up with are the ones Eq. 13's totals in
Tab. 1 are made of (l layers at the full count, L - l at the reduced one)."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl
from tests.path_check import LOGIT_TOL, assert_flips_in_margin, bits_f64, check_att, dev_bits, host_bits, keep_flips

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


@pytest.mark.parametrize("l_dense,L", [(2, 5), (0, 3), (3, 3)])
def test_stack_with_dense_leading_layers_against_the_oracle(l_dense, L):
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[3].scaled(B=3, n_layers=L, n_gen=9)
    B, H, D, dt = cfg.B, cfg.n_heads, cfg.head_dim, cfg.dtype
    n_vis, k_vis, n_text = 96, 24, 10
    T = n_vis + n_text
    cap_dense, cap = 128, 64                                    # two capacities: full rows and reduced rows
    scale = 1.0 / np.sqrt(D)
    tdt = wl.torch_dtype(dt)
    D_ = lambda x: wl.to_torch(x, dt, DEV)

    p_img, p_txt = wl.make_predictor(cfg, "img"), wl.make_predictor(cfg, "txt")
    x_vis = wl.host_normal(cfg, wl.S_X_VIS, (B, n_vis, cfg.hidden))
    k_src = [wl.host_normal(cfg, wl.S_K, (B, T, H, D), sub=l) for l in range(L)]
    v_src = [wl.host_normal(cfg, wl.S_V, (B, T, H, D), sub=l) for l in range(L)]
    x_dec = wl.host_normal(cfg, wl.S_X_TXT, (cfg.n_gen, B, cfg.hidden))
    q_dec, k_dec, v_dec = (wl.host_normal(cfg, s, (cfg.n_gen, L, B, H, D)) for s in (wl.S_DEC_Q, wl.S_DEC_K, wl.S_DEC_V))

    ctx = dl.Context(cfg.hidden, H, D, cfg.pred_hidden, tdt, 0, max_batch=B, max_rows=B * n_vis, cap=cap_dense)
    pred = lambda p: dl.Predictor(D_(p.w1), torch.from_numpy(p.b1).to(DEV), torch.from_numpy(p.w2).to(DEV), p.b2)
    pi, pt = pred(p_img), pred(p_txt)
    i32 = dict(dtype=torch.int32, device=DEV)

    # ---- the decision (taken once, after layer l) and the two kinds of caches
    score = torch.empty(B, n_vis, dtype=torch.float32, device=DEV)
    kept_idx = torch.empty(B, k_vis, **i32)
    keep = torch.empty(B, n_vis, dtype=torch.uint8, device=DEV)
    n_vis_d, k_d = torch.full((B,), n_vis, **i32), torch.full((B,), k_vis, **i32)
    ctx.prefill_select(pi, D_(x_vis), n_vis_d, k_d, score, kept_idx, keep)
    keep_gpu = keep.cpu().numpy()
    idx_iso, keep_iso = orc.prefill_select(score.cpu().numpy().astype(np.float64), np.full(B, n_vis, np.int32),
                                           np.full(B, k_vis, np.int32), k_vis)
    assert np.array_equal(keep_iso, keep_gpu)
    all_rows = torch.ones(B, n_vis, dtype=torch.uint8, device=DEV)
    t_src = np.full(B, T, np.int32)
    t_src_d = torch.from_numpy(t_src).to(DEV)
    len_dense, cache_len = torch.zeros(B, **i32), torch.zeros(B, **i32)
    caps = [cap_dense if l < l_dense else cap for l in range(L)]
    k_cache = [torch.zeros(B, H, caps[l], D, dtype=tdt, device=DEV) for l in range(L)]
    v_cache = [torch.zeros(B, H, caps[l], D, dtype=tdt, device=DEV) for l in range(L)]
    for l in range(L):
        dense = l < l_dense
        last = (l == l_dense - 1) if dense else (l == L - 1)
        ctx.compact_kv(D_(k_src[l]), D_(v_src[l]), all_rows if dense else keep, t_src_d, k_cache[l], v_cache[l],
                       len_dense if dense else cache_len, commit=last)
    # oracle state
    udt = np.uint32 if dt == "f32" else np.uint16
    o_k = [np.zeros((B, H, caps[l], D), udt) for l in range(L)]
    o_v = [np.zeros((B, H, caps[l], D), udt) for l in range(L)]
    masks = {True: np.ones((B, T), np.uint8), False: np.ones((B, T), np.uint8)}
    masks[False][:, :n_vis] = keep_gpu
    o_len = {True: np.zeros(B, np.int32), False: np.zeros(B, np.int32)}
    for l in range(L):
        dense = l < l_dense
        ln = np.zeros(B, np.int32)
        st, _ = orc.append_rows(host_bits(k_src[l], dt), host_bits(v_src[l], dt), masks[dense], t_src, o_k[l], o_v[l], ln)
        assert st == orc.OK
        o_len[dense] = ln
    if l_dense > 0:
        assert np.array_equal(len_dense.cpu().numpy(), o_len[True]) and list(o_len[True]) == [T] * B
    if l_dense < L:
        assert np.array_equal(cache_len.cpu().numpy(), o_len[False]) and list(o_len[False]) == [k_vis + n_text] * B

    # ---- the accounting the split stands for: Eq. 13 per layer at each layer's own image-token count
    width = 4096
    img_tokens = [n_vis if l < l_dense else int(keep_gpu[0].sum()) for l in range(L)]
    assert sum(orc.prefill_flops(1, n, width) for n in img_tokens) == \
        orc.prefill_flops_model(L, l_dense, n_vis, k_vis, width)

    # ---- decode steps over the stack
    logit = torch.empty(B, dtype=torch.float32, device=DEV)
    keep_t = torch.empty(B, dtype=torch.uint8, device=DEV)
    out_t = torch.empty(L, B, H, D, dtype=tdt, device=DEV)
    kept_total = 0
    for t in range(cfg.n_gen):
        ctx.decode_step_stack(pt, D_(x_dec[t]), logit, keep_t, k_cache, v_cache, l_dense, cap_dense, cap,
                              len_dense if l_dense > 0 else None, cache_len if l_dense < L else None,
                              D_(q_dec[t]), D_(k_dec[t]), D_(v_dec[t]), scale, out_t)
        z_gpu, m_gpu, o_gpu = logit.cpu().numpy(), keep_t.cpu().numpy(), wl.from_torch(out_t)
        z_ref = orc.predictor_logits(x_dec[t], p_txt.w1, p_txt.b1, p_txt.w2, p_txt.b2)
        assert float(np.abs(z_gpu - z_ref).max()) <= LOGIT_TOL
        assert np.array_equal(m_gpu, orc.decode_keep(z_gpu.astype(np.float64)))
        assert_flips_in_margin(keep_flips(z_ref, m_gpu), f"keep (step {t})")
        for l in range(L):
            n_l = o_len[l < l_dense]
            ref = np.empty((B, H, D))
            for b in range(B):
                for h in range(H):
                    ref[b, h] = orc.attention_decode_compact(
                        q_dec[t, l, b, h], k_dec[t, l, b, h], v_dec[t, l, b, h], bits_f64(o_k[l][b, h, : n_l[b]], dt),
                        bits_f64(o_v[l][b, h, : n_l[b]], dt), int(n_l[b]), scale)
            check_att(o_gpu[l], ref, f"decode attention step {t} layer {l}")
        new_len = {}
        for l in range(L):
            dense = l < l_dense
            ln = o_len[dense].copy()
            decision = np.ones(B, np.uint8) if dense else m_gpu
            st, _ = orc.append_rows(host_bits(k_dec[t, l], dt)[:, None], host_bits(v_dec[t, l], dt)[:, None],
                                    decision[:, None], None, o_k[l], o_v[l], ln)
            assert st == orc.OK
            new_len[dense] = ln
        o_len.update(new_len)
        kept_total += int(m_gpu.sum())
        if l_dense > 0:
            assert np.array_equal(len_dense.cpu().numpy(), o_len[True]), f"dense lengths after step {t}"
        if l_dense < L:
            assert np.array_equal(cache_len.cpu().numpy(), o_len[False]), f"compact lengths after step {t}"
    # every dense layer has grown by one row per step, every later layer by the kept tokens only
    if l_dense > 0:
        assert list(o_len[True]) == [T + cfg.n_gen] * B
    if l_dense < L:
        assert int(o_len[False].sum()) == B * (k_vis + n_text) + kept_total
    for l in range(L):
        gk, gv = dev_bits(k_cache[l]), dev_bits(v_cache[l])
        n_l = o_len[l < l_dense]
        for b in range(B):
            assert np.array_equal(gk[b, :, : n_l[b]], o_k[l][b, :, : n_l[b]]), f"K cache layer {l} seq {b}"
            assert np.array_equal(gv[b, :, : n_l[b]], o_v[l][b, :, : n_l[b]]), f"V cache layer {l} seq {b}"
    assert ctx.device_status()[0] == dl.DL_OK
    ctx.close()
