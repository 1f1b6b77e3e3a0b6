"""GPU parity of the 8-bit K/V cache extension (not in the paper) against oracle/fp8_cache.py: the stored bytes are
compared bit for bit, the attention output within the bf16 path's tolerances against the oracle ON THE SAME BYTES;
what quantisation itself costs against the unquantised oracle is printed, not bounded."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from oracle import fp8_cache as f8
from paper_2412_00876_b200 import workloads as wl
from tests.path_check import att_errors, check_att

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def _setup(B, H, cap, seed):
    from paper_2412_00876_b200 import binding as dl
    D = 128
    rng = np.random.default_rng(seed)
    ctx = dl.Context(256, H, D, 64, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
    r = lambda *shape: wl.round_to_storage(rng.normal(0, 1, shape).astype(np.float32), "bf16")
    return dl, ctx, rng, r, D


def test_quantise_is_bit_exact():
    B, H, cap = 3, 4, 80
    dl, ctx, rng, r, D = _setup(B, H, cap, 1)
    src = r(B, H, cap, D)
    src[0, 0, 0, :8] = [0.0, -0.0, 1e-4, -1e-4, 500.0, -500.0, 0.0625, 3.0]       # zeros, tiny, clamped values
    scale = np.array([0.01, 0.05, 0.5, 2.0 ** -6], np.float32)
    lens = np.array([80, 17, 0], np.int32)
    dst = torch.full((B, H, cap, D), 0xAB, dtype=torch.uint8, device=DEV)
    ctx.quantize_kv_fp8(wl.to_torch(src, "bf16", DEV), torch.from_numpy(lens).to(DEV), torch.from_numpy(scale).to(DEV), dst)
    got = dst.cpu().numpy()
    ref = f8.quantize_rows(src, scale[None, :, None, None])
    for b in range(B):
        assert np.array_equal(got[b, :, : lens[b]], ref[b, :, : lens[b]]), f"sequence {b}"
        assert np.all(got[b, :, lens[b]:] == 0xAB)                    # rows past the length are not written
    assert ctx.device_status()[0] == 0
    ctx.close()


@pytest.mark.parametrize("B,H,cap,lens", [(4, 4, 320, [0, 1, 31, 300]), (2, 8, 1408, [1300, 777]),
                                           (5, 2, 128, [32, 33, 64, 100, 127])])
def test_decode_attention_and_append_over_the_byte_cache(B, H, cap, lens):
    """Ragged lengths over several 32-row tiles and split sequences; kept tokens are appended as bytes."""
    dl, ctx, rng, r, D = _setup(B, H, cap, 7 + B)
    lens = np.array(lens, np.int32)
    k_src, v_src = r(B, H, cap, D), r(B, H, cap, D)
    k_scale = (np.abs(k_src).max(axis=(0, 2, 3)) / 448.0 * rng.uniform(1.0, 1.5, H)).astype(np.float32)
    v_scale = (np.abs(v_src).max(axis=(0, 2, 3)) / 448.0 * rng.uniform(1.0, 1.5, H)).astype(np.float32)
    q, kt, vt = r(B, H, D), r(B, H, D), r(B, H, D)
    keep = (np.arange(B) % 2 == 0).astype(np.uint8)
    ln = torch.from_numpy(lens).to(DEV)
    kc = torch.zeros(B, H, cap, D, dtype=torch.uint8, device=DEV)
    vc = torch.zeros(B, H, cap, D, dtype=torch.uint8, device=DEV)
    ks_d, vs_d = torch.from_numpy(k_scale).to(DEV), torch.from_numpy(v_scale).to(DEV)
    ctx.quantize_kv_fp8(wl.to_torch(k_src, "bf16", DEV), ln, ks_d, kc)
    ctx.quantize_kv_fp8(wl.to_torch(v_src, "bf16", DEV), ln, vs_d, vc)
    # rows past the lengths hold bytes that decode to NaN: they must never reach a result
    for b in range(B):
        kc[b, :, lens[b]:] = 0x7F
        vc[b, :, lens[b]:] = 0xFF
    o_k = f8.quantize_rows(k_src, k_scale[None, :, None, None])
    o_v = f8.quantize_rows(v_src, v_scale[None, :, None, None])
    scale = 1.0 / np.sqrt(D)
    out = torch.zeros(B, H, D, dtype=torch.bfloat16, device=DEV)
    ctx.sparse_attn_decode_fp8(wl.to_torch(q, "bf16", DEV), wl.to_torch(kt, "bf16", DEV), wl.to_torch(vt, "bf16", DEV),
                               kc, vc, ks_d, vs_d, ln, torch.from_numpy(keep).to(DEV), scale, out)
    got = wl.from_torch(out)
    gk, gv = kc.cpu().numpy(), vc.cpu().numpy()
    ref = np.empty((B, H, D))
    plain = np.empty((B, H, D))
    for b in range(B):
        n = int(lens[b])
        for h in range(H):
            ref[b, h] = f8.attention_decode_fp8(q[b, h], kt[b, h], vt[b, h], o_k[b, h], o_v[b, h], k_scale[h], v_scale[h], n, scale)
            plain[b, h] = orc.attention_decode_compact(q[b, h], kt[b, h], vt[b, h], k_src[b, h].astype(np.float64),
                                                       v_src[b, h].astype(np.float64), n, scale)
            # the cache below the length is untouched; a kept token's row is the oracle's bytes
            assert np.array_equal(gk[b, h, :n], o_k[b, h, :n]) and np.array_equal(gv[b, h, :n], o_v[b, h, :n])
            if keep[b] and n < cap:
                assert np.array_equal(gk[b, h, n], f8.quantize_rows(kt[b, h], k_scale[h])), f"appended K row {b},{h}"
                assert np.array_equal(gv[b, h, n], f8.quantize_rows(vt[b, h], v_scale[h])), f"appended V row {b},{h}"
            elif n < cap:
                assert np.all(gk[b, h, n] == 0x7F) and np.all(gv[b, h, n] == 0xFF)
    check_att(got, ref, "fp8 decode attention against the oracle on the same bytes")
    mx, rl = att_errors(got, plain)
    print(f"cost of quantisation against the unquantised oracle: max-abs {mx:.3e}, relative L2 {rl:.3e}")
    assert ctx.device_status()[0] == 0
    ctx.close()


def test_full_cache_is_left_untouched_and_reported():
    B, H, cap = 2, 2, 64
    dl, ctx, rng, r, D = _setup(B, H, cap, 3)
    lens = torch.tensor([cap, 10], dtype=torch.int32, device=DEV)
    kc = torch.full((B, H, cap, D), 0x38, dtype=torch.uint8, device=DEV)
    vc = torch.full((B, H, cap, D), 0x38, dtype=torch.uint8, device=DEV)
    one = torch.ones(H, dtype=torch.float32, device=DEV)
    t = lambda x: wl.to_torch(x, "bf16", DEV)
    out = torch.zeros(B, H, D, dtype=torch.bfloat16, device=DEV)
    before = kc.clone()
    ctx.sparse_attn_decode_fp8(t(r(B, H, D)), t(r(B, H, D)), t(r(B, H, D)), kc, vc, one, one, lens,
                               torch.ones(B, dtype=torch.uint8, device=DEV), 0.1, out)
    torch.cuda.synchronize()
    assert torch.equal(kc[0], before[0])
    code, detail = ctx.device_status()
    assert code == dl.DL_ERR_CAPACITY and detail == 0
    ctx.close()


def test_full_size_launch_on_sampled_heads():
    """The launch bench.py times (`--micro decode_fp8`, config 3: B = 32, H = 32, cap 1344, lengths 784 +- 16, every
    sequence kept), checked on sampled (sequence, head) pairs the oracle recomputes one by one, plus what holds at
    any size: bytes below the lengths untouched, appended rows equal to the oracle's bytes."""
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[3]
    B, H, D, cap = cfg.B, cfg.n_heads, cfg.head_dim, cfg.cap
    g = torch.Generator(device=DEV).manual_seed(33)
    mk = lambda: (torch.randint(0, 0x7E, (B, H, cap, D), dtype=torch.uint8, device=DEV, generator=g) |
                  (torch.randint(0, 2, (B, H, cap, D), dtype=torch.uint8, device=DEV, generator=g) << 7))
    kc, vc = mk(), mk()
    k0, v0 = kc.clone(), vc.clone()
    rng = np.random.default_rng(4)
    lens = np.clip(784 + rng.integers(-16, 17, B), 0, cap - 1).astype(np.int32)
    ks = rng.uniform(1 / 96, 1 / 48, H).astype(np.float32)
    vs = rng.uniform(1 / 96, 1 / 48, H).astype(np.float32)
    r = lambda *shape: wl.round_to_storage(rng.normal(0, 1, shape).astype(np.float32), "bf16")
    q, kt, vt = r(B, H, D), r(B, H, D), r(B, H, D)
    t = lambda x: wl.to_torch(x, "bf16", DEV)
    ctx = dl.Context(cfg.hidden, H, D, cfg.pred_hidden, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
    out = torch.zeros(B, H, D, dtype=torch.bfloat16, device=DEV)
    scale = 1.0 / np.sqrt(D)
    ctx.sparse_attn_decode_fp8(t(q), t(kt), t(vt), kc, vc, torch.from_numpy(ks).to(DEV), torch.from_numpy(vs).to(DEV),
                               torch.from_numpy(lens).to(DEV), torch.ones(B, dtype=torch.uint8, device=DEV), scale, out)
    got = wl.from_torch(out)
    pairs = [(0, 0), (B - 1, H - 1)] + [(int(rng.integers(0, B)), int(rng.integers(0, H))) for _ in range(14)]
    for b, h in pairs:
        n = int(lens[b])
        ck, cv = k0[b, h].cpu().numpy(), v0[b, h].cpu().numpy()
        ref = f8.attention_decode_fp8(q[b, h], kt[b, h], vt[b, h], ck, cv, ks[h], vs[h], n, scale)
        check_att(got[b, h][None], ref[None], f"fp8 decode attention, full size, b={b} h={h}")
        assert np.array_equal(kc[b, h, n].cpu().numpy(), f8.quantize_rows(kt[b, h], ks[h]))
        assert np.array_equal(vc[b, h, n].cpu().numpy(), f8.quantize_rows(vt[b, h], vs[h]))
    # nothing but row lens[b] of each (b, h) has changed
    rows = torch.arange(cap, device=DEV)[None, None, :, None]
    untouched = rows != torch.from_numpy(lens).to(DEV).long()[:, None, None, None]
    assert torch.equal(torch.where(untouched, kc, 0), torch.where(untouched, k0, 0))
    assert torch.equal(torch.where(untouched, vc, 0), torch.where(untouched, v0, 0))
    assert ctx.device_status()[0] == 0
    ctx.close()


@pytest.mark.parametrize("B,H,L,cap", [(32, 32, 4, 512), (3, 4, 5, 320)])
def test_layer_stack_over_byte_caches_equals_per_layer_calls(B, H, L, cap):
    """L overlapped launches (one CTA slot per SM each at the large shape, split sequences sharing the scratch sets
    in rotation at the small one) give bit for bit what separate calls give, every time, and the lengths advance
    once behind the last layer."""
    from paper_2412_00876_b200 import binding as dl
    D = 128
    g = torch.Generator(device=DEV).manual_seed(5)
    mk = lambda: (torch.randint(0, 0x7E, (B, H, cap, D), dtype=torch.uint8, device=DEV, generator=g) |
                  (torch.randint(0, 2, (B, H, cap, D), dtype=torch.uint8, device=DEV, generator=g) << 7))
    base_k, base_v = [mk() for _ in range(L)], [mk() for _ in range(L)]
    rng = np.random.default_rng(6)
    r = lambda *shape: wl.to_torch(wl.round_to_storage(rng.normal(0, 1, shape).astype(np.float32), "bf16"), "bf16", DEV)
    q, kt, vt = r(L, B, H, D), r(L, B, H, D), r(L, B, H, D)
    ks = torch.from_numpy(rng.uniform(1 / 96, 1 / 48, (L, H)).astype(np.float32)).to(DEV)
    vs = torch.from_numpy(rng.uniform(1 / 96, 1 / 48, (L, H)).astype(np.float32)).to(DEV)
    lens = rng.integers(0, cap, B).astype(np.int32)
    keep = torch.from_numpy((np.arange(B) % 3 != 0).astype(np.uint8)).to(DEV)
    ctx = dl.Context(256, H, D, 64, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
    scale = 1 / np.sqrt(D)
    results = []
    for mode in ("per-layer", "stack", "stack", "stack"):
        kc, vc = [t.clone() for t in base_k], [t.clone() for t in base_v]
        ln = torch.from_numpy(lens).to(DEV)
        out = torch.zeros(L, B, H, D, dtype=torch.bfloat16, device=DEV)
        if mode == "per-layer":
            for l in range(L):
                ctx.sparse_attn_decode_fp8(q[l], kt[l], vt[l], kc[l], vc[l], ks[l], vs[l], ln, keep, scale, out[l])
            ctx.commit_len(keep, ln, cap)
        else:
            ctx.sparse_attn_decode_fp8_layers(q, kt, vt, kc, vc, ks, vs, ln, keep, scale, out, commit=True)
        torch.cuda.synchronize()
        results.append((out, kc, vc, ln.cpu().numpy()))
    ref = results[0]
    assert np.array_equal(ref[3], lens + (keep.cpu().numpy() != 0) * (lens < cap))
    for out, kc, vc, ln in results[1:]:
        assert torch.equal(out.view(torch.int16), ref[0].view(torch.int16))
        assert np.array_equal(ln, ref[3])
        for l in range(L):
            assert torch.equal(kc[l], ref[1][l]) and torch.equal(vc[l], ref[2][l])
    assert ctx.device_status()[0] == 0
    ctx.close()
