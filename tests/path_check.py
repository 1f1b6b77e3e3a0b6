"""Runs the whole path on the GPU through the C ABI, step by step beside the CPU oracle,
and checks every stage: predictor logits, selection, compaction, prefill attention, then
decode steps (keep decision, attention with the current token, conditional append).

Used by the GPU tests and by the smoke check.  Tolerances are the ones the project states:
  logits            max-abs 1e-2 (bf16 inputs, fp32 accumulation)
  attention outputs max-abs 2e-2 and relative L2 5e-3
  masks, indices, cache contents and lengths: bit-exact
  a keep / select decision may differ from the oracle's only where the oracle's margin is
  below 1e-3; every such flip is logged and the oracle then continues with the GPU's decision.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import binding as dl
from paper_2412_00876_b200 import workloads as wl

LOGIT_TOL = 1e-2
ATT_MAXABS = 2e-2
ATT_RELL2 = 5e-3
MARGIN = 1e-3
# The paper-architecture predictors are a chain of ten bf16 tensor-core layers (activations rounded to bf16
# between them), whose decision values are only required, and only able, to meet the logit tolerance: two values
# each within LOGIT_TOL can change order when the oracle's gap is below twice that.
MARGIN_CHAIN = 2 * LOGIT_TOL


def dev_bits(t: torch.Tensor) -> np.ndarray:
    """Raw storage of a device tensor as a numpy unsigned array."""
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.contiguous().view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def host_bits(x_f32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(x_f32, dtype=np.float32).view(np.uint32)
    return wl.f32_to_bf16_bits(x_f32)


def bits_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return bits.view(np.float32).astype(np.float64)
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def att_errors(got: np.ndarray, ref: np.ndarray):
    d = got - ref
    return float(np.abs(d).max()) if d.size else 0.0, float(np.linalg.norm(d) / max(np.linalg.norm(ref), 1e-30))


def check_att(got, ref, what):
    mx, rl = att_errors(got, ref)
    assert mx <= ATT_MAXABS and rl <= ATT_RELL2, f"{what}: max-abs {mx:.3e} rel-L2 {rl:.3e}"
    return mx, rl


def selection_flips(s_ref: np.ndarray, keep_gpu: np.ndarray, k: int, margin: float = MARGIN):
    """Tokens whose GPU selection differs from the oracle's, with the oracle margin check."""
    _, keep_ref = orc.topk_select(s_ref, k)
    diff = np.flatnonzero(keep_ref != keep_gpu)
    if len(diff) == 0:
        return []
    order = np.sort(s_ref)[::-1]
    lo = order[k] if k < len(order) else -np.inf          # best score the oracle drops
    hi = order[k - 1] if k > 0 else np.inf                # worst score the oracle keeps
    flips = []
    for i in diff:
        # a token the oracle keeps may be dropped only if it is within the margin of the best dropped score;
        # a token the oracle drops may be kept only if it is within the margin of the worst kept score
        ok = (s_ref[i] - lo < margin) if keep_ref[i] else (hi - s_ref[i] < margin)
        flips.append((int(i), float(s_ref[i]), bool(ok)))
    return flips


def keep_flips(z_ref: np.ndarray, keep_gpu: np.ndarray, threshold: float = 0.0):
    """Decode decisions that differ from the oracle's, each with whether the oracle's logit lies inside the margin."""
    m_ref = orc.decode_keep(z_ref, threshold)
    return [(int(b), float(z_ref[b]), bool(abs(z_ref[b] - threshold) < MARGIN)) for b in np.flatnonzero(m_ref != keep_gpu)]


def assert_flips_in_margin(flips, what: str):
    """The rule for decisions that floating point takes: a flip is tolerated (and logged by the caller) only where
    the oracle's margin is below MARGIN; anything else is a failure."""
    for f in flips:
        assert f[-1], f"{what} flip outside the margin: {f}"


def run_chained(cid: int, n_decode: int | None = None, B: int | None = None, L: int | None = None,
                ragged: bool = False, options: dict | None = None, device: int = 0, verbose: bool = False,
                shape: dict | None = None, txt_keep_rate: float | None = None):
    """`shape` overrides fields of the configuration (n_vis, k_vis, n_text, ...); `txt_keep_rate` moves the decode
    predictor's second-layer bias so that about that share of this run's generated tokens gets a positive logit
    (the bias is an input of both implementations; it is taken from the oracle's logits of the same rows)."""
    cfg = wl.CONFIGS[cid]
    kw = dict(shape or {})
    if B is not None:
        kw["B"] = B
    if L is not None:
        kw["n_layers"] = L
    if n_decode is not None:
        kw["n_gen"] = n_decode
    cfg = cfg.scaled(**kw)
    B, L, H, D, dt = cfg.B, cfg.n_layers, cfg.n_heads, cfg.head_dim, cfg.dtype
    T = cfg.n_vis + cfg.n_text
    cap = cfg.cap
    dev = torch.device("cuda", device)
    scale = 1.0 / np.sqrt(D)
    report = {"config": cfg.name, "flips": []}

    # ------------------------------------------------------------------ inputs (host)
    p_img = wl.make_predictor(cfg, "img")
    p_txt = wl.make_predictor(cfg, "txt")
    x_vis = wl.host_normal(cfg, wl.S_X_VIS, (B, cfg.n_vis, cfg.hidden))
    q_src = [wl.host_normal(cfg, wl.S_Q, (B, T, H, D), sub=l) for l in range(L)]
    k_src = [wl.host_normal(cfg, wl.S_K, (B, T, H, D), sub=l) for l in range(L)]
    v_src = [wl.host_normal(cfg, wl.S_V, (B, T, H, D), sub=l) for l in range(L)]
    n_text = wl.ragged_text_lengths(cfg) if ragged else np.full(B, cfg.n_text, np.int32)
    n_vis = np.full(B, cfg.n_vis, np.int32)
    k_arr = np.full(B, cfg.k_vis, np.int32)
    if ragged and B > 1:
        n_vis[1] = cfg.n_vis - 5
        k_arr[1] = min(cfg.k_vis, n_vis[1]) // 2
    t_src = (cfg.n_vis + n_text).astype(np.int32)
    x_dec = wl.host_normal(cfg, wl.S_X_TXT, (cfg.n_gen, B, cfg.hidden))
    if txt_keep_rate is not None:
        z0 = orc.predictor_logits(x_dec.reshape(-1, cfg.hidden), p_txt.w1, p_txt.b1, p_txt.w2, 0.0)
        p_txt = wl.make_predictor(cfg, "txt", b2=float(-np.quantile(z0, 1.0 - txt_keep_rate)))
    q_dec = wl.host_normal(cfg, wl.S_DEC_Q, (cfg.n_gen, L, B, H, D))
    k_dec = wl.host_normal(cfg, wl.S_DEC_K, (cfg.n_gen, L, B, H, D))
    v_dec = wl.host_normal(cfg, wl.S_DEC_V, (cfg.n_gen, L, B, H, D))

    def D_(x):
        return wl.to_torch(x, dt, dev)

    def pred_dev(p):
        return dl.Predictor(D_(p.w1), torch.from_numpy(p.b1).to(dev), torch.from_numpy(p.w2).to(dev), p.b2)

    ctx = dl.Context(cfg.hidden, H, D, cfg.pred_hidden, wl.torch_dtype(dt), device, max_batch=B,
                     max_rows=B * cfg.n_vis, cap=cap)
    for o, v in (options or {}).items():
        ctx.set_option(o, v)
    pi, pt = pred_dev(p_img), pred_dev(p_txt)
    i32 = dict(dtype=torch.int32, device=dev)

    # ------------------------------------------------------------------ a1 + a2: prefill select
    score = torch.empty(B, cfg.n_vis, dtype=torch.float32, device=dev)
    k_max = int(k_arr.max())
    kept_idx = torch.empty(B, k_max, **i32)
    keep = torch.empty(B, cfg.n_vis, dtype=torch.uint8, device=dev)
    n_vis_d, k_d = torch.from_numpy(n_vis).to(dev), torch.from_numpy(k_arr).to(dev)
    ctx.prefill_select(pi, D_(x_vis), n_vis_d, k_d, score, kept_idx, keep)
    s_gpu = score.cpu().numpy()
    keep_gpu, idx_gpu = keep.cpu().numpy(), kept_idx.cpu().numpy()
    s_ref = orc.predictor_logits(x_vis, p_img.w1, p_img.b1, p_img.w2, p_img.b2)
    report["score_maxabs"] = float(np.abs(s_gpu - s_ref).max())
    assert report["score_maxabs"] <= LOGIT_TOL, report
    # stage-isolated: the GPU's selection is the oracle's selection of the GPU's own fp32 scores
    idx_iso, keep_iso = orc.prefill_select(s_gpu.astype(np.float64), n_vis, k_arr, k_max)
    assert np.array_equal(keep_iso, keep_gpu) and np.array_equal(idx_iso, idx_gpu), "top-k not bit-exact"
    assert list(keep_gpu.sum(axis=1)) == list(k_arr)
    # chained: decisions may differ from the fp64 oracle's only inside the margin
    for b in range(B):
        fl = selection_flips(s_ref[b, : n_vis[b]], keep_gpu[b, : n_vis[b]], int(k_arr[b]))
        report["flips"] += [("select", b, i, s) for (i, s, _) in fl]
        assert_flips_in_margin(fl, f"selection (sequence {b})")

    # ------------------------------------------------------------------ a3: compaction (K, V, Q per layer)
    cache_len = torch.zeros(B, **i32)
    t_src_d = torch.from_numpy(t_src).to(dev)
    tdt = wl.torch_dtype(dt)
    k_cache = [torch.zeros(B, H, cap, D, dtype=tdt, device=dev) for _ in range(L)]
    v_cache = [torch.zeros(B, H, cap, D, dtype=tdt, device=dev) for _ in range(L)]
    q_cache = [torch.zeros(B, H, cap, D, dtype=tdt, device=dev) for _ in range(L)]
    for l in range(L):
        ctx.compact_kv(D_(k_src[l]), D_(v_src[l]), keep, t_src_d, k_cache[l], v_cache[l], cache_len, commit=False)
        ctx.compact_kv(D_(q_src[l]), None, keep, t_src_d, q_cache[l], None, cache_len, commit=(l == L - 1))
    # oracle, with the GPU's (already checked) mask
    udt = np.uint32 if dt == "f32" else np.uint16
    o_len = np.zeros(B, np.int32)
    o_k = [np.zeros((B, H, cap, D), udt) for _ in range(L)]
    o_v = [np.zeros((B, H, cap, D), udt) for _ in range(L)]
    o_q = [np.zeros((B, H, cap, D), udt) for _ in range(L)]
    mask = np.ones((B, T), np.uint8)
    mask[:, : cfg.n_vis] = keep_gpu
    for l in range(L):
        ln = o_len.copy()
        st, _ = orc.append_rows(host_bits(k_src[l], dt), host_bits(v_src[l], dt), mask, t_src, o_k[l], o_v[l], ln)
        assert st == orc.OK
        ln2 = o_len.copy()
        orc.append_rows(host_bits(q_src[l], dt), host_bits(q_src[l], dt), mask, t_src, o_q[l], o_q[l].copy(), ln2)
    o_len = ln
    assert np.array_equal(cache_len.cpu().numpy(), o_len), "cache_len after prefill"
    assert list(o_len) == list(k_arr + n_text)

    def caches_equal(tag):
        for l in range(L):
            gk, gv = dev_bits(k_cache[l]), dev_bits(v_cache[l])
            for b in range(B):
                n = o_len[b]
                assert np.array_equal(gk[b, :, :n], o_k[l][b, :, :n]), f"{tag}: K cache layer {l} seq {b}"
                assert np.array_equal(gv[b, :, :n], o_v[l][b, :, :n]), f"{tag}: V cache layer {l} seq {b}"

    caches_equal("prefill")
    for l in range(L):
        gq = dev_bits(q_cache[l])
        for b in range(B):
            assert np.array_equal(gq[b, :, : o_len[b]], o_q[l][b, :, : o_len[b]])

    # ------------------------------------------------------------------ a4: prefill attention
    n_max = int(o_len.max())
    worst = (0.0, 0.0)
    for l in range(L):
        out = torch.zeros(B, n_max, H, D, dtype=tdt, device=dev)
        ctx.sparse_attn_prefill(q_cache[l], k_cache[l], v_cache[l], cache_len, n_max, scale, out)
        got = wl.from_torch(out)
        for b in range(B):
            n = int(o_len[b])
            ref = np.stack([orc.attention_prefill_compact(bits_f64(o_q[l][b, h], dt), bits_f64(o_k[l][b, h], dt),
                                                          bits_f64(o_v[l][b, h], dt), n, scale)
                            for h in range(H)], axis=1)          # [n, H, D]
            e = check_att(got[b, :n], ref, f"prefill attention layer {l} seq {b}")
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
    report["prefill_att_maxabs"], report["prefill_att_rel_l2"] = worst

    # ------------------------------------------------------------------ a5-a7: decode steps
    logit = torch.empty(B, dtype=torch.float32, device=dev)
    keep_t = torch.empty(B, dtype=torch.uint8, device=dev)
    out_t = torch.empty(L, B, H, D, dtype=tdt, device=dev)
    kp, vp = ctx.pointer_array(k_cache), ctx.pointer_array(v_cache)
    worst = (0.0, 0.0)
    logit_err = 0.0
    kept_total = 0
    for t in range(cfg.n_gen):
        ctx.decode_step(pt, D_(x_dec[t]), logit, keep_t, D_(q_dec[t]), D_(k_dec[t]), D_(v_dec[t]), kp, vp, L, cap,
                        cache_len, scale, out_t)
        z_gpu, m_gpu, o_gpu = logit.cpu().numpy(), keep_t.cpu().numpy(), wl.from_torch(out_t)
        z_ref = orc.predictor_logits(x_dec[t], p_txt.w1, p_txt.b1, p_txt.w2, p_txt.b2)
        logit_err = max(logit_err, float(np.abs(z_gpu - z_ref).max()))
        assert logit_err <= LOGIT_TOL, f"decode logit error {logit_err}"
        assert np.array_equal(m_gpu, orc.decode_keep(z_gpu.astype(np.float64))), "keep flag vs own logit"
        fl = keep_flips(z_ref, m_gpu)
        report["flips"] += [("keep", b, t, z) for (b, z, _) in fl]
        assert_flips_in_margin(fl, f"keep (step {t})")
        for l in range(L):
            ref = np.empty((B, H, D))
            for b in range(B):
                for h in range(H):
                    ref[b, h] = orc.attention_decode_compact(
                        q_dec[t, l, b, h], k_dec[t, l, b, h], v_dec[t, l, b, h],
                        bits_f64(o_k[l][b, h, : o_len[b]], dt), bits_f64(o_v[l][b, h, : o_len[b]], dt),
                        int(o_len[b]), scale)
            e = check_att(o_gpu[l], ref, f"decode attention step {t} layer {l}")
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        for l in range(L):
            ln = o_len.copy()
            st, _ = orc.append_rows(host_bits(k_dec[t, l], dt)[:, None], host_bits(v_dec[t, l], dt)[:, None],
                                    m_gpu[:, None], None, o_k[l], o_v[l], ln)
            assert st == orc.OK
        o_len = ln if L > 0 else o_len + m_gpu
        kept_total += int(m_gpu.sum())
        assert np.array_equal(cache_len.cpu().numpy(), o_len), f"cache_len after step {t}"
    caches_equal("decode")
    report["decode_logit_maxabs"] = logit_err
    report["decode_att_maxabs"], report["decode_att_rel_l2"] = worst
    report["decode_kept"] = f"{kept_total}/{cfg.n_gen * B}"
    code, detail = ctx.device_status()
    assert code == dl.DL_OK, f"device status {code} detail {detail}"
    ctx.close()
    if verbose:
        print(report)
    return report
