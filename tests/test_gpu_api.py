"""C-ABI behaviour on the GPU: argument checks return error codes (nothing traps), the layer-stack
call equals per-layer calls bit for bit, and a decode step is reproducible."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2412_00876_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_invalid_arguments_are_refused_with_codes():
    from paper_2412_00876_b200 import binding as dl
    lib = dl.lib()
    h = C.c_void_p()
    bad = dl.ModelDesc(4096, 32, 96, 1024, dl.DL_BF16)                 # head_dim 96 is not built
    assert lib.dl_create(C.byref(h), 0, C.byref(bad)) == dl.DL_ERR_UNSUPPORTED
    assert lib.dl_create(C.byref(h), 99, C.byref(dl.ModelDesc(4096, 32, 128, 1024, dl.DL_BF16))) == dl.DL_ERR_CUDA
    ctx = dl.Context(256, 4, 128, 64, torch.bfloat16, 0, max_batch=2, max_rows=8, cap=64)
    t = torch.zeros(2 * 4 * 64 * 128 + 8, dtype=torch.bfloat16, device=DEV)
    ln = torch.zeros(2, dtype=torch.int32, device=DEV)
    p = t.data_ptr()
    # NULL tensor, misaligned tensor, cap beyond the workspace, batch beyond the workspace
    assert lib.dl_sparse_attn_decode(ctx._h, None, p, p, p, p, ln.data_ptr(), None, 2, 64, 0.1, p, None) == dl.DL_ERR_INVALID_ARG
    assert lib.dl_sparse_attn_decode(ctx._h, p + 2, p, p, p, p, ln.data_ptr(), None, 2, 64, 0.1, p, None) == dl.DL_ERR_ALIGNMENT
    assert lib.dl_sparse_attn_decode(ctx._h, p, p, p, p, p, ln.data_ptr(), None, 2, 128, 0.1, p, None) == dl.DL_ERR_WORKSPACE
    assert lib.dl_sparse_attn_decode(ctx._h, p, p, p, p, p, ln.data_ptr(), None, 3, 64, 0.1, p, None) == dl.DL_ERR_WORKSPACE
    assert lib.dl_sparse_attn_prefill(ctx._h, p, p, p, ln.data_ptr(), 2, 64, 65, 0.1, p, None) == dl.DL_ERR_INVALID_ARG   # n_max > cap
    assert lib.dl_sparse_attn_prefill(ctx._h, p, p, p, ln.data_ptr(), 2, 64, 64, -1.0, p, None) == dl.DL_ERR_INVALID_ARG  # scale <= 0
    assert lib.dl_compact_kv(ctx._h, p, p, None, 0, None, 2, 4, p, None, 64, ln.data_ptr(), 1, None) == dl.DL_ERR_INVALID_ARG  # v_src without v_cache
    assert lib.dl_set_option(ctx._h, 77, 1) == dl.DL_ERR_INVALID_ARG
    assert lib.dl_topk_from_scores(ctx._h, p, None, ln.data_ptr(), 1, 20000, None, 0, p, None) == dl.DL_ERR_UNSUPPORTED
    # empty problems are fine
    assert lib.dl_sparse_attn_decode(ctx._h, None, None, None, None, None, None, None, 0, 64, 0.1, None, None) == dl.DL_OK
    assert ctx.device_status()[0] == 0
    ctx.close()


@pytest.mark.parametrize("B,H,L,cap", [
    (32, 32, 3, 512),      # 1024 (b,h) pairs: unsplit launches, two layers side by side
    (8, 32, 8, 1024),      # 256 pairs: every sequence split in four, more layers than scratch sets
    (2, 32, 5, 2048),      # 64 pairs: fewer items per chunk than SMs in places, split, both CTA slots
])
def test_layer_stack_equals_per_layer_calls_and_is_reproducible(B, H, L, cap):
    """A stack of layers issued as one call (launches that overlap on the GPU, sharing the split scratch in
    rotation) gives bit for bit what separate per-layer calls give, every time."""
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[3]
    D = 128
    ctx = dl.Context(256, H, D, 64, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
    mk = lambda s, shape, sub=0: wl.device_normal(cfg, s, shape, DEV, sub=sub)
    q, kt, vt = mk(wl.S_DEC_Q, (L, B, H, D)), mk(wl.S_DEC_K, (L, B, H, D)), mk(wl.S_DEC_V, (L, B, H, D))
    base_k = [mk(wl.S_CACHE_K, (B, H, cap, D), l) for l in range(L)]
    base_v = [mk(wl.S_CACHE_V, (B, H, cap, D), l) for l in range(L)]
    ln = torch.from_numpy(wl.host_rng(3, wl.S_LEN).integers(0, cap, B).astype(np.int32)).to(DEV)
    keep = torch.from_numpy((np.arange(B) % 3 != 0).astype(np.uint8)).to(DEV)
    scale = 1 / np.sqrt(D)
    results = []
    for mode in ("per-layer", "stack", "stack", "stack", "stack"):
        kc, vc = [t.clone() for t in base_k], [t.clone() for t in base_v]
        out = torch.zeros(L, B, H, D, dtype=torch.bfloat16, device=DEV)
        if mode == "per-layer":
            for l in range(L):
                ctx.sparse_attn_decode(q[l], kt[l], vt[l], kc[l], vc[l], ln, keep, scale, out[l])
        else:
            ctx.sparse_attn_decode_layers(q, kt, vt, ctx.pointer_array(kc), ctx.pointer_array(vc), L, cap, ln, keep,
                                          scale, out)
        torch.cuda.synchronize()
        results.append((out, kc, vc))
    ref = results[0]
    for out, kc, vc in results[1:]:
        assert torch.equal(out.view(torch.int16), ref[0].view(torch.int16))
        for l in range(L):
            assert torch.equal(kc[l].view(torch.int16), ref[1][l].view(torch.int16))
            assert torch.equal(vc[l].view(torch.int16), ref[2][l].view(torch.int16))
    assert ctx.device_status()[0] == 0
    ctx.close()


def test_pipelined_host_fed_steps_equal_single_host_steps():
    """dl_decode_steps_host (copies of step t+1 and t-1 overlapping the compute of step t) leaves the same
    caches, lengths, outputs and keep flags as one dl_decode_step_host call per step."""
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[2]
    B, H, D, L, cap, hidden, ph, n_steps = 4, 4, 128, 3, 128, 256, 64, 7
    rng = np.random.default_rng(5)
    w1 = torch.from_numpy(rng.normal(0, 0.05, (ph, hidden)).astype(np.float32)).to(torch.bfloat16).to(DEV)
    pd = dl.Predictor(w1, torch.zeros(ph, device=DEV), torch.from_numpy(rng.normal(0, 0.5, ph).astype(np.float32)).to(DEV), 0.0)
    pin = lambda t: t.cpu().pin_memory()
    xs = [pin(torch.randn(B, hidden).to(torch.bfloat16)) for _ in range(n_steps)]
    qs, ks, vs = ([pin(torch.randn(L, B, H, D).to(torch.bfloat16)) for _ in range(n_steps)] for _ in range(3))
    base_k = [torch.randn(B, H, cap, D, device=DEV).to(torch.bfloat16) for _ in range(L)]
    base_v = [torch.randn(B, H, cap, D, device=DEV).to(torch.bfloat16) for _ in range(L)]
    scale = 1 / np.sqrt(D)
    results = []
    for mode in ("single", "pipelined"):
        ctx = dl.Context(hidden, H, D, ph, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
        kc, vc = [t.clone() for t in base_k], [t.clone() for t in base_v]
        kp, vp = ctx.pointer_array(kc), ctx.pointer_array(vc)
        ln = torch.tensor([5, 0, 60, 100], dtype=torch.int32, device=DEV)
        outs = [pin(torch.zeros(L, B, H, D, dtype=torch.bfloat16)) for _ in range(n_steps)]
        keeps = [pin(torch.zeros(B, dtype=torch.uint8)) for _ in range(n_steps)]
        two = lambda *shape, dt=torch.bfloat16: torch.empty((2,) + shape, dtype=dt, device=DEV)
        sx, sq, sk, sv, so = two(B, hidden), two(L, B, H, D), two(L, B, H, D), two(L, B, H, D), two(L, B, H, D)
        lg, kd = two(B, dt=torch.float32), two(B, dt=torch.uint8)
        if mode == "single":
            for t in range(n_steps):
                ctx.decode_step_host(pd, xs[t], qs[t], ks[t], vs[t], outs[t], keeps[t], sx[0], sq[0], sk[0], sv[0],
                                     so[0], lg[0], kd[0], kp, vp, L, cap, ln, scale)
        else:
            ctx.decode_steps_host(pd, xs, qs, ks, vs, outs, keeps, sx, sq, sk, sv, so, lg, kd, kp, vp, L, cap, ln, scale)
        torch.cuda.synchronize()
        assert ctx.device_status()[0] == 0
        results.append((outs, keeps, kc, vc, ln.cpu()))
        ctx.close()
    a, b = results
    assert any(int(k.sum()) not in (0, B) for k in a[1]), "keep flags should vary"
    for t in range(n_steps):
        assert torch.equal(a[0][t].view(torch.int16), b[0][t].view(torch.int16)), f"step {t} output"
        assert torch.equal(a[1][t], b[1][t])
    for l in range(L):
        assert torch.equal(a[2][l].view(torch.int16), b[2][l].view(torch.int16))
        assert torch.equal(a[3][l].view(torch.int16), b[3][l].view(torch.int16))
    assert torch.equal(a[4], b[4])



def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """The library's wait routine on a barrier that never completes (a dedicated self-test kernel: no copy in
    flight, nothing to drain): it gives up after its bound, DL_ERR_TIMEOUT reaches the status word, the call
    returns well within a second and the next kernels of the same context work."""
    import time
    from paper_2412_00876_b200 import binding as dl
    ctx = dl.Context(256, 4, 128, 64, torch.bfloat16, 0, max_batch=4, max_rows=4, cap=128)
    t0 = time.perf_counter()
    ctx.selftest_wait_timeout(polls=200)
    code, detail = ctx.device_status()                    # synchronises
    assert time.perf_counter() - t0 < 1.0
    assert code == dl.DL_ERR_TIMEOUT and detail == 0x5E1F
    assert ctx.device_status()[0] == 0                    # reading clears it
    logit = torch.tensor([1.0, -1.0, 0.0, 2.0], device="cuda:0")
    keep = torch.empty(4, dtype=torch.uint8, device="cuda:0")
    ctx.decode_keep(None, None, logit, keep)
    assert keep.cpu().tolist() == [1, 0, 0, 1] and ctx.device_status()[0] == 0
    ctx.close()
