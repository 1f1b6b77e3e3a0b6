"""dl_sparse_attn_decode_static: decode attention for callers that cannot allocate device memory.

Some users of this library run where a cudaMalloc is not an option: inside a serving engine that
owns all device memory through its own pool, in a plugin that only ever receives buffers, or on a
GPU that is already filled to the brim.  They cannot hand the library a workspace, so this entry
point keeps the kernel's scratch in a fixed array inside the library.  The test calls it through
the C ABI twice in a row (the array keeps the first call's contents, so the second call shows that
what must start at zero is cleared) and compares with the workspace-based entry point.

Collected last on purpose: a failure here cannot hide the other tests in a stop-at-first-failure run.
"""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl
from tests import path_check as pc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(B, H, D, cap, seed):
    cfg = wl.CONFIGS[2]
    mk = lambda s, shape: wl.to_torch(wl.host_normal(cfg, s, shape, sub=seed), "bf16", DEV)
    return (mk(wl.S_DEC_Q, (B, H, D)), mk(wl.S_DEC_K, (B, H, D)), mk(wl.S_DEC_V, (B, H, D)),
            mk(wl.S_CACHE_K, (B, H, cap, D)), mk(wl.S_CACHE_V, (B, H, cap, D)))


def test_static_scratch_variant_matches_workspace_variant_twice():
    from paper_2412_00876_b200 import binding as dl
    B, H, D, cap = 4, 8, 128, 1024
    lens = [0, 300, 777, 1024]                      # none, two chunks, four chunks, a full cache
    ctx = dl.Context(256, H, D, 64, torch.bfloat16, 0, max_batch=B, max_rows=B, cap=cap)
    scale = 1 / np.sqrt(D)
    ln = torch.tensor(lens, dtype=torch.int32, device=DEV)
    keep = torch.tensor([1, 0, 1, 0], dtype=torch.uint8, device=DEV)
    for call in range(2):                            # two calls in a row, different data
        q, kt, vt, kc, vc = _inputs(B, H, D, cap, seed=10 + call)
        kc2, vc2 = kc.clone(), vc.clone()
        ref = torch.zeros(B, H, D, dtype=torch.bfloat16, device=DEV)
        got = torch.zeros_like(ref)
        ctx.sparse_attn_decode(q, kt, vt, kc, vc, ln, keep, scale, ref)
        ctx.sparse_attn_decode_static(q, kt, vt, kc2, vc2, ln, keep, scale, got)
        torch.cuda.synchronize()
        mx, rl = pc.att_errors(wl.from_torch(got), wl.from_torch(ref))
        assert mx <= pc.ATT_MAXABS and rl <= pc.ATT_RELL2, (call, mx, rl)
        assert torch.equal(kc.view(torch.int16), kc2.view(torch.int16))      # same fused append
        assert torch.equal(vc.view(torch.int16), vc2.view(torch.int16))
    assert ctx.device_status()[0] == 0
    ctx.close()


def test_static_scratch_variant_refuses_problems_beyond_its_array():
    from paper_2412_00876_b200 import binding as dl
    B, H, D, cap = 512, 32, 128, 4096                # 512*32 (b,h) pairs * 2 slots * 130 floats = 17 MB > 8 MiB
    ctx = dl.Context(256, H, D, 64, torch.bfloat16, 0, max_batch=1, max_rows=1, cap=64)
    t = torch.zeros(16, dtype=torch.bfloat16, device=DEV)          # never dereferenced: the call is refused
    ln = torch.zeros(B, dtype=torch.int32, device=DEV)
    st = dl.lib().dl_sparse_attn_decode_static(ctx._h, t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(),
                                               t.data_ptr(), ln.data_ptr(), None, B, cap, 0.1, t.data_ptr(), None)
    assert st == dl.DL_ERR_WORKSPACE
    ctx.close()


def _raw_context(hidden, H, D, pred, dtype_code):
    """A context made through the bare C ABI with NO workspace: what a caller that cannot allocate has."""
    import ctypes as C
    from paper_2412_00876_b200 import binding as dl
    h = C.c_void_p()
    desc = dl.ModelDesc(hidden, H, D, pred, dtype_code)
    assert dl.lib().dl_create(C.byref(h), 0, C.byref(desc)) == dl.DL_OK
    return h


@pytest.mark.parametrize("dtype,H,D,lens,cap", [("bf16", 4, 128, [0, 5, 200, 640], 640), ("f32", 8, 64, [3, 0, 131, 64], 192)])
def test_static_scratch_variant_without_any_workspace_matches_the_oracle(dtype, H, D, lens, cap):
    """No dl_set_workspace at all (no status word either): outputs against the CPU oracle, the fused append, and a
    full cache with keep = 1, which must leave the cache untouched and still return DL_OK."""
    from paper_2412_00876_b200 import binding as dl
    B = len(lens)
    cfg = wl.CONFIGS[2]
    mk = lambda s, shape: wl.host_normal(cfg, s, shape, sub=77, dtype=dtype)
    q, kt, vt = mk(wl.S_DEC_Q, (B, H, D)), mk(wl.S_DEC_K, (B, H, D)), mk(wl.S_DEC_V, (B, H, D))
    kc, vc = mk(wl.S_CACHE_K, (B, H, cap, D)), mk(wl.S_CACHE_V, (B, H, cap, D))
    T = lambda x: wl.to_torch(x, dtype, DEV)
    qd, ktd, vtd, kcd, vcd = T(q), T(kt), T(vt), T(kc), T(vc)
    before_k, before_v = kcd.clone(), vcd.clone()
    ln = torch.tensor(lens, dtype=torch.int32, device=DEV)
    keep = torch.ones(B, dtype=torch.uint8, device=DEV)
    out = torch.zeros(B, H, D, dtype=wl.torch_dtype(dtype), device=DEV)
    scale = 1 / np.sqrt(D)
    h = _raw_context(256, H, D, 64, dl.DL_BF16 if dtype == "bf16" else dl.DL_F32)
    for _ in range(2):
        st = dl.lib().dl_sparse_attn_decode_static(h, qd.data_ptr(), ktd.data_ptr(), vtd.data_ptr(), kcd.data_ptr(),
                                                   vcd.data_ptr(), ln.data_ptr(), keep.data_ptr(), B, cap, float(scale),
                                                   out.data_ptr(), None)
        assert st == dl.DL_OK
        torch.cuda.synchronize()
        got = wl.from_torch(out)
        for b in range(B):
            ref = np.stack([orc.attention_decode_compact(q[b, hh], kt[b, hh], vt[b, hh], kc[b, hh], vc[b, hh], lens[b], scale)
                            for hh in range(H)])
            pc.check_att(got[b], ref, f"static decode, no workspace, seq {b}")
        for b in range(B):
            n = lens[b]
            if n < cap:                                             # appended at row n, nothing else touched
                assert torch.equal(kcd[b, :, n], ktd[b]) and torch.equal(vcd[b, :, n], vtd[b])
                kcd[b, :, n] = before_k[b, :, n]
                vcd[b, :, n] = before_v[b, :, n]
        assert torch.equal(kcd, before_k) and torch.equal(vcd, before_v)   # incl. the full cache: unchanged
    assert dl.lib().dl_destroy(h) == dl.DL_OK
