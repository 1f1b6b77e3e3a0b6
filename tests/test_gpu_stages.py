"""Stage-isolated GPU-vs-oracle parity through the C ABI: every kernel is fed inputs from
the seeded generators (or the oracle's upstream output) and compared element by element."""
import numpy as np
import pytest
import torch

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl
from tests import path_check as pc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ctx(dtype="bf16", H=4, D=128, hidden=256, pred=64, B=4, rows=0, cap=512):
    from paper_2412_00876_b200 import binding as dl
    return dl.Context(hidden, H, D, pred, wl.torch_dtype(dtype), 0, max_batch=B, max_rows=max(rows, B), cap=cap)


# ------------------------------------------------------------------------------ top-k
def _topk_case(score, n_vis, k):
    ctx = _ctx(B=score.shape[0])
    B, n = score.shape
    k_max = max(1, int(np.max(k)))
    s_d = torch.from_numpy(score.astype(np.float32)).to(DEV)
    idx = torch.full((B, k_max), -7, dtype=torch.int32, device=DEV)
    keep = torch.full((B, n), 9, dtype=torch.uint8, device=DEV)
    nv = None if n_vis is None else torch.from_numpy(np.asarray(n_vis, np.int32)).to(DEV)
    ctx.topk_from_scores(s_d, nv, torch.from_numpy(np.asarray(k, np.int32)).to(DEV), idx, keep)
    ridx, rkeep = orc.prefill_select(score.astype(np.float32).astype(np.float64), n_vis, np.asarray(k), k_max)
    assert np.array_equal(keep.cpu().numpy(), rkeep)
    assert np.array_equal(idx.cpu().numpy(), ridx)
    return ctx


def test_topk_random_ties_and_sizes():
    rng = np.random.default_rng(0)
    for n in (1, 31, 144, 576, 2880, 5000, 16384):
        B = 3
        score = np.round(rng.normal(size=(B, n)), 1 if n < 3000 else 3)      # many exact ties
        k = np.array([0, n, n // 4])
        _topk_case(score, None, k)
        n_vis = np.array([n, max(1, n // 2), max(1, n - 1)])
        k = np.array([n // 5, max(1, n // 2), 1])
        _topk_case(score, n_vis, k)


def test_topk_special_values():
    s = np.array([[0.0, -0.0, 0.0, -0.0, 1.0, -1.0, np.inf, -np.inf],
                  [np.nan, 1.0, np.nan, -np.inf, 2.0, 2.0, 2.0, -0.0],
                  [5.0] * 8])
    for k in ([2, 3, 4], [8, 8, 8], [0, 0, 0], [5, 7, 1]):
        ctx = _topk_case(s, None, np.array(k))
    code, _ = ctx.device_status()
    from paper_2412_00876_b200 import binding as dl
    assert code == dl.DL_WARN_NAN


def test_decisions_inside_the_margin_flip_are_logged_and_followed():
    """Host-made scores whose fp64 order at the selection boundary differs from their fp32 order (the two boundary
    scores round to one fp32 value, so the GPU keeps the lower index) and logits that are positive in fp64 but
    zero in fp32: the checker must report these flips as inside the margin, and the compaction that follows is
    compared with the oracle run on the GPU's decisions."""
    from paper_2412_00876_b200 import binding as dl
    rng = np.random.default_rng(11)
    B, n, k, H, D = 2, 64, 8, 4, 128
    s64 = rng.normal(size=(B, n))
    for b in range(B):
        order = np.argsort(-s64[b])
        lo_i, hi_i = sorted((int(order[k - 1]), int(order[k])))      # the boundary pair, lower index first
        base = float(np.float32(s64[b, order[k]]))
        s64[b, lo_i], s64[b, hi_i] = base, base + 1e-10              # fp64: the higher index wins; fp32: a tie
    ctx = _ctx(B=B, cap=128)
    idx = torch.empty(B, k, dtype=torch.int32, device=DEV)
    keep = torch.empty(B, n, dtype=torch.uint8, device=DEV)
    ctx.topk_from_scores(torch.from_numpy(s64.astype(np.float32)).to(DEV), None,
                         torch.full((B,), k, dtype=torch.int32, device=DEV), idx, keep)
    keep_gpu = keep.cpu().numpy()
    n_flips = 0
    for b in range(B):
        fl = pc.selection_flips(s64[b], keep_gpu[b], k)
        assert len(fl) == 2, fl                                      # one token in, one out
        pc.assert_flips_in_margin(fl, "selection")
        n_flips += len(fl)
    assert n_flips == 2 * B
    # downstream, with the GPU's decision: compaction equals the oracle's filtered copy under the GPU's mask
    cfg = wl.CONFIGS[2]
    src = wl.host_normal(cfg, wl.S_K, (B, n, H, D))
    kc = torch.zeros(B, H, 128, D, dtype=torch.bfloat16, device=DEV)
    ln = torch.zeros(B, dtype=torch.int32, device=DEV)
    ctx.compact_kv(wl.to_torch(src, "bf16", DEV), None, keep, torch.full((B,), n, dtype=torch.int32, device=DEV), kc,
                   None, ln, commit=True)
    o_k = np.zeros((B, H, 128, D), np.uint16)
    o_len = np.zeros(B, np.int32)
    orc.append_rows(pc.host_bits(src, "bf16"), pc.host_bits(src, "bf16"), keep_gpu, None, o_k, o_k.copy(), o_len)
    assert list(ln.cpu().numpy()) == list(o_len) == [k] * B
    assert np.array_equal(pc.dev_bits(kc)[:, :, :k], o_k[:, :, :k])
    # decode keep: logits given (x = NULL); 1e-50 is +0 in fp32
    z64 = np.array([0.3, 1e-50, -0.4, 2e-46], dtype=np.float64)
    logit = torch.from_numpy(z64.astype(np.float32)).to(DEV)
    kt = torch.empty(4, dtype=torch.uint8, device=DEV)
    ctx4 = _ctx(B=4)
    ctx4.decode_keep(None, None, logit, kt)
    fl = pc.keep_flips(z64, kt.cpu().numpy())
    assert [b for b, _, _ in fl] == [1, 3]
    pc.assert_flips_in_margin(fl, "keep")


def test_topk_paper_rate():
    rng = np.random.default_rng(1)
    k = orc.k_from_rate(576, 20, 100)
    _topk_case(rng.normal(size=(2, 576)), None, np.array([k, k]))


# ------------------------------------------------------------------------------ compaction
@pytest.mark.parametrize("impl", [0, 1, 2])         # library's choice; register-staged; bulk copy by even row ranges
@pytest.mark.parametrize("dtype,H,D", [("bf16", 32, 128), ("f32", 8, 64), ("bf16", 3, 64), ("f32", 2, 128)])
def test_compaction_bit_exact(dtype, H, D, impl):
    from paper_2412_00876_b200 import binding as dl
    rng = np.random.default_rng(2)
    B, T, nv, cap = 3, 150, 110, 256
    cfg = wl.CONFIGS[1]
    ctx = _ctx(dtype, H, D, B=B, cap=cap)
    ctx.set_option(dl.DL_OPT_COMPACT_IMPL, impl)
    ks = wl.host_normal(cfg, wl.S_K, (B, T, H, D), dtype=dtype)
    vs = wl.host_normal(cfg, wl.S_V, (B, T, H, D), dtype=dtype)
    keep = (rng.random((B, nv)) < 0.3).astype(np.uint8)
    keep[1] = wl.static_keep_pattern("structure", nv)
    keep[2] = 0
    t_src = np.array([T, T - 17, nv + 3], np.int32)
    start = np.array([0, 5, 40], np.int32)
    tdt = wl.torch_dtype(dtype)
    kc = torch.zeros(B, H, cap, D, dtype=tdt, device=DEV)
    vc = torch.zeros_like(kc)
    ln = torch.from_numpy(start.copy()).to(DEV)
    ctx.compact_kv(wl.to_torch(ks, dtype, DEV), wl.to_torch(vs, dtype, DEV), torch.from_numpy(keep).to(DEV),
                   torch.from_numpy(t_src).to(DEV), kc, vc, ln, commit=True)
    udt = np.uint32 if dtype == "f32" else np.uint16
    ok, ov = np.zeros((B, H, cap, D), udt), np.zeros((B, H, cap, D), udt)
    oln = start.copy()
    mask = np.ones((B, T), np.uint8)
    mask[:, :nv] = keep
    st, _ = orc.append_rows(pc.host_bits(ks, dtype), pc.host_bits(vs, dtype), mask, t_src, ok, ov, oln)
    assert st == orc.OK
    assert np.array_equal(ln.cpu().numpy(), oln)
    gk, gv = pc.dev_bits(kc), pc.dev_bits(vc)
    for b in range(B):
        assert np.array_equal(gk[b, :, start[b]:oln[b]], ok[b, :, start[b]:oln[b]])
        assert np.array_equal(gv[b, :, start[b]:oln[b]], ov[b, :, start[b]:oln[b]])
        assert not gk[b, :, oln[b]:].any() and not gk[b, :, :start[b]].any()      # nothing written elsewhere
    assert ctx.device_status()[0] == 0


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("n_tensors", [1, 5, 8])
def test_compaction_of_several_tensors_under_one_decision(n_tensors, impl):
    """dl_compact_kv_layers (one plan, a run of overlapped copy launches): bit for bit what the oracle's filtered copy
    gives for every tensor and what single calls give, nothing written outside the appended rows, the length committed
    once; a sequence that does not fit is left untouched in every tensor."""
    from paper_2412_00876_b200 import binding as dl
    rng = np.random.default_rng(40 + n_tensors)
    dtype, H, D, B, T, nv, cap = "bf16", 8, 128, 4, 200, 160, 192
    cfg = wl.CONFIGS[2]
    ctx = _ctx(dtype, H, D, B=B, cap=cap)
    ctx.set_option(dl.DL_OPT_COMPACT_IMPL, impl)
    srcs = [wl.host_normal(cfg, wl.S_K, (B, T, H, D), sub=i) for i in range(n_tensors)]
    keep = (rng.random((B, nv)) < 0.25).astype(np.uint8)
    keep[3] = 1                                                   # 160 + 40 text rows > what is left of the cache
    t_src = np.array([T, T - 9, nv, T], np.int32)
    start = np.array([0, 7, 30, 20], np.int32)
    fill = 0x4242
    caches = [torch.full((B, H, cap, D), 0, dtype=torch.int16, device=DEV).fill_(fill).view(torch.bfloat16) for _ in range(n_tensors)]
    ln = torch.from_numpy(start.copy()).to(DEV)
    keep_d, t_d = torch.from_numpy(keep).to(DEV), torch.from_numpy(t_src).to(DEV)
    ctx.compact_kv_layers([wl.to_torch(x, dtype, DEV) for x in srcs], caches, keep_d, t_d, ln, commit=True)
    code, detail = ctx.device_status()
    assert code == dl.DL_ERR_CAPACITY and detail == 3
    mask = np.ones((B, T), np.uint8)
    mask[:, :nv] = keep
    o_len = None
    for i in range(n_tensors):
        o_c = np.full((B, H, cap, D), fill, np.uint16)
        o_len = start.copy()
        st, _ = orc.append_rows(pc.host_bits(srcs[i], dtype), pc.host_bits(srcs[i], dtype), mask, t_src, o_c, o_c.copy(), o_len)
        assert st == orc.ERR_CAPACITY
        assert np.array_equal(pc.dev_bits(caches[i]), o_c), f"tensor {i}"     # every byte, appended or not
    assert list(ln.cpu().numpy()) == list(o_len) and o_len[3] == start[3]
    # the same through single calls
    singles = [torch.full((B, H, cap, D), 0, dtype=torch.int16, device=DEV).fill_(fill).view(torch.bfloat16) for _ in range(n_tensors)]
    ln2 = torch.from_numpy(start.copy()).to(DEV)
    for i in range(n_tensors):
        ctx.compact_kv(wl.to_torch(srcs[i], dtype, DEV), None, keep_d, t_d, singles[i], None, ln2, commit=(i == n_tensors - 1))
    for i in range(n_tensors):
        assert torch.equal(singles[i].view(torch.int16), caches[i].view(torch.int16))
    assert torch.equal(ln, ln2)
    ctx.device_status()


@pytest.mark.parametrize("impl", [1, 2])
def test_compaction_does_not_read_a_stale_plan(impl):
    """The copy kernel starts while the plan kernel of the same call still runs.  With the workspace holding
    a hostile old plan (count -1 = skip the sequence) a copy that read the plan too early would leave rows
    unwritten: both copy kernels, several calls in a row, on a grid large enough to start early."""
    from paper_2412_00876_b200 import binding as dl
    B, T, H, D, nv, cap = 16, 704, 32, 128, 576, 768
    ctx = dl.Context(4096, H, D, 1024, torch.bfloat16, 0, max_batch=B, max_rows=B * nv, cap=cap)
    ctx.set_option(dl.DL_OPT_COMPACT_IMPL, impl)
    g = torch.Generator(device=DEV).manual_seed(7)
    ks = torch.randn(B, T, H, D, device=DEV, generator=g).to(torch.bfloat16)
    vs = torch.randn(B, T, H, D, device=DEV, generator=g).to(torch.bfloat16)
    keep = (torch.rand(B, nv, device=DEV, generator=g) < 0.25).to(torch.uint8)
    t_src = torch.full((B,), T, dtype=torch.int32, device=DEV)
    for rep in range(4):
        ctx._ws.fill_(0xFF)                                  # every plan word reads -1 until rewritten
        base = (ctx._ws.data_ptr() + 255) // 256 * 256       # same memory set up again: status and tickets zeroed
        n = dl.lib().dl_workspace_bytes(ctx._h, B, B * nv, cap)
        assert dl.lib().dl_set_workspace(ctx._h, base, n, B, B * nv, cap, None) == 0
        kc = torch.zeros(B, H, cap, D, dtype=torch.bfloat16, device=DEV)
        vc = torch.zeros(B, H, cap, D, dtype=torch.bfloat16, device=DEV)
        ln = torch.zeros(B, dtype=torch.int32, device=DEV)
        ctx.compact_kv(ks, vs, keep, t_src, kc, vc, ln, commit=True)
        torch.cuda.synchronize()
        for b in range(B):
            rows = torch.cat([torch.nonzero(keep[b]).flatten(), torch.arange(nv, T, device=DEV)])
            assert int(ln[b]) == rows.numel()
            for src, got in ((ks, kc), (vs, vc)):
                ref = src[b, rows].permute(1, 0, 2)
                assert torch.equal(ref.view(torch.int16), got[b, :, : rows.numel()].view(torch.int16)), (rep, b)
        assert ctx.device_status()[0] == 0
    ctx.close()


def test_compaction_from_pinned_host_sources():
    """dl_compact_kv_host (the kernel reads the kept rows from pinned host memory) gives the caches and lengths
    of dl_compact_kv on a device copy of the same sources, bit for bit; pageable memory is refused."""
    from paper_2412_00876_b200 import binding as dl
    B, T, H, D, nv, cap = 4, 300, 32, 128, 200, 320
    ctx = dl.Context(4096, H, D, 1024, torch.bfloat16, 0, max_batch=B, max_rows=B * nv, cap=cap)
    g = torch.Generator().manual_seed(11)
    ks_h = torch.randn(B, T, H, D, generator=g).to(torch.bfloat16).pin_memory()
    vs_h = torch.randn(B, T, H, D, generator=g).to(torch.bfloat16).pin_memory()
    keep = (torch.rand(B, nv, generator=g) < 0.3).to(torch.uint8).to(DEV)
    t_src = torch.tensor([T, T - 9, nv, 5], dtype=torch.int32, device=DEV)
    res = []
    for host in (False, True):
        kc = torch.zeros(B, H, cap, D, dtype=torch.bfloat16, device=DEV)
        vc = torch.zeros_like(kc)
        ln = torch.tensor([0, 3, 0, 1], dtype=torch.int32, device=DEV)
        if host:
            ctx.compact_kv_host(ks_h, vs_h, keep, t_src, kc, vc, ln, commit=True)
        else:
            ctx.compact_kv(ks_h.to(DEV), vs_h.to(DEV), keep, t_src, kc, vc, ln, commit=True)
        torch.cuda.synchronize()
        res.append((kc, vc, ln))
    assert torch.equal(res[0][2], res[1][2]) and int(res[0][2].sum()) > 0
    assert torch.equal(res[0][0].view(torch.int16), res[1][0].view(torch.int16))
    assert torch.equal(res[0][1].view(torch.int16), res[1][1].view(torch.int16))
    assert ctx.device_status()[0] == 0
    with pytest.raises(dl.DlError) as e:                       # pageable host memory: not reachable from the device
        ctx.compact_kv_host(torch.zeros(B, T, H, D, dtype=torch.bfloat16), None, keep, t_src, res[0][0], None, res[0][2])
    assert e.value.code == dl.DL_ERR_INVALID_ARG
    ctx.close()


def test_compaction_keep_all_single_tensor_and_capacity():
    from paper_2412_00876_b200 import binding as dl
    B, T, H, D, cap = 2, 40, 4, 128, 48
    cfg = wl.CONFIGS[2]
    ctx = _ctx("bf16", H, D, B=B, cap=cap)
    ks = wl.host_normal(cfg, wl.S_K, (B, T, H, D))
    kc = torch.zeros(B, H, cap, D, dtype=torch.bfloat16, device=DEV)
    ln = torch.tensor([0, 20], dtype=torch.int32, device=DEV)          # sequence 1: 20 + 40 > 48
    ctx.compact_kv(wl.to_torch(ks, "bf16", DEV), None, None, None, kc, None, ln, commit=True)
    assert list(ln.cpu().numpy()) == [T, 20]
    g = pc.dev_bits(kc)
    assert np.array_equal(g[0, :, :T], pc.host_bits(ks, "bf16")[0].transpose(1, 0, 2))
    assert not g[1].any()
    code, detail = ctx.device_status()
    assert code == dl.DL_ERR_CAPACITY and detail == 1
    assert ctx.device_status()[0] == 0                                 # reading clears it


# ------------------------------------------------------------------------------ predictor
@pytest.mark.parametrize("cid,rows", [(1, 144), (2, 576), (2, 7), (4, 33)])
def test_predictor_scores(cid, rows):
    from paper_2412_00876_b200 import binding as dl
    cfg = wl.CONFIGS[cid]
    p = wl.make_predictor(cfg, "img")
    x = wl.host_normal(cfg, wl.S_X_VIS, (rows, cfg.hidden))
    ctx = dl.Context(cfg.hidden, cfg.n_heads, cfg.head_dim, cfg.pred_hidden, wl.torch_dtype(cfg.dtype), 0,
                     max_batch=1, max_rows=rows, cap=64)
    pd = dl.Predictor(wl.to_torch(p.w1, cfg.dtype, DEV), torch.from_numpy(p.b1).to(DEV),
                      torch.from_numpy(p.w2).to(DEV), p.b2)
    ref = orc.predictor_logits(x, p.w1, p.b1, p.w2, p.b2)
    for impl in (1, 2):
        out = torch.zeros(rows, dtype=torch.float32, device=DEV)
        ctx.set_option(dl.DL_OPT_PREDICTOR_IMPL, impl)
        try:
            ctx.predictor_scores(pd, wl.to_torch(x, cfg.dtype, DEV), out)
        except dl.DlError as e:
            assert impl == 2 and e.code == dl.DL_ERR_UNSUPPORTED
            continue
        err = float(np.abs(out.cpu().numpy() - ref).max())
        assert err <= pc.LOGIT_TOL, (impl, err)
        assert err <= 2e-4, (impl, err)          # fp32 accumulation is far inside the tolerance


# ------------------------------------------------------------------------------ decode attention
def _decode_case(dtype, H, D, lens, cap, chunk=0, with_keep=True, seed=0):
    from paper_2412_00876_b200 import binding as dl
    B = len(lens)
    cfg = wl.CONFIGS[2]
    ctx = _ctx(dtype, H, D, B=B, cap=cap)
    if chunk:
        ctx.set_option(dl.DL_OPT_DECODE_CHUNK, chunk)
    kc = wl.host_normal(cfg, wl.S_CACHE_K, (B, H, cap, D), dtype=dtype, sub=seed)
    vc = wl.host_normal(cfg, wl.S_CACHE_V, (B, H, cap, D), dtype=dtype, sub=seed)
    q = wl.host_normal(cfg, wl.S_DEC_Q, (B, H, D), dtype=dtype, sub=seed)
    kt = wl.host_normal(cfg, wl.S_DEC_K, (B, H, D), dtype=dtype, sub=seed)
    vt = wl.host_normal(cfg, wl.S_DEC_V, (B, H, D), dtype=dtype, sub=seed)
    keep = (np.arange(B) % 2).astype(np.uint8)
    scale = 1 / np.sqrt(D)
    tdt = wl.torch_dtype(dtype)
    for b in range(B):                          # rows past the length are unspecified: make them hostile
        kc[b, :, lens[b]:] = np.nan
        vc[b, :, lens[b]:] = np.nan
    kc_d, vc_d = wl.to_torch(kc, dtype, DEV), wl.to_torch(vc, dtype, DEV)
    ek0, ev0 = pc.dev_bits(kc_d).copy(), pc.dev_bits(vc_d).copy()      # cache contents before the calls
    ln = torch.tensor(lens, dtype=torch.int32, device=DEV)
    outs = []
    for rep in range(2):
        out = torch.zeros(B, H, D, dtype=tdt, device=DEV)
        ctx.sparse_attn_decode(wl.to_torch(q, dtype, DEV), wl.to_torch(kt, dtype, DEV), wl.to_torch(vt, dtype, DEV),
                               kc_d, vc_d, ln, torch.from_numpy(keep).to(DEV) if with_keep else None, scale, out)
        outs.append(out)
    assert torch.equal(outs[0].view(torch.uint8), outs[1].view(torch.uint8)), "not reproducible"
    got = wl.from_torch(outs[0])
    ref = np.empty((B, H, D))
    for b in range(B):
        for h in range(H):
            ref[b, h] = orc.attention_decode_compact(q[b, h], kt[b, h], vt[b, h], kc[b, h], vc[b, h], lens[b], scale)
    pc.check_att(got, ref, f"decode {dtype} D={D} lens={lens}")
    # the append: kept sequences have (k_t, v_t) at row len, everything else is untouched
    gk, gv = pc.dev_bits(kc_d), pc.dev_bits(vc_d)
    ek, ev = ek0, ev0
    full = False
    for b in range(B):
        if with_keep and keep[b]:
            if lens[b] < cap:
                ek[b, :, lens[b]] = pc.host_bits(kt, dtype)[b]
                ev[b, :, lens[b]] = pc.host_bits(vt, dtype)[b]
            else:
                full = True
    assert np.array_equal(gk, ek) and np.array_equal(gv, ev)
    assert list(ln.cpu().numpy()) == list(lens)
    code, _ = ctx.device_status()
    assert code == (dl.DL_ERR_CAPACITY if full else 0)


def test_decode_attention_lengths_and_chunks():
    _decode_case("bf16", 4, 128, [0, 1, 7, 8, 9, 63, 64, 65], cap=128)
    _decode_case("bf16", 4, 128, [255, 256, 257, 300, 511, 512, 640, 1], cap=640)            # several chunks
    _decode_case("bf16", 2, 128, [64, 65, 129, 448, 449, 3], cap=512, chunk=64)             # many chunks
    _decode_case("bf16", 32, 128, [336, 208, 700, 0, 1000], cap=1024, seed=1)                # more items than SMs
    _decode_case("bf16", 2, 128, [100, 128], cap=128)                                        # full cache + keep


def test_decode_attention_other_types():
    _decode_case("f32", 8, 64, [0, 68, 132, 5], cap=192)
    _decode_case("f32", 2, 128, [100, 300], cap=320)
    _decode_case("bf16", 4, 64, [100, 300, 64], cap=320, with_keep=False)


# ------------------------------------------------------------------------------ prefill attention
def _prefill_case(dtype, H, D, lens, amp=1.0):
    from paper_2412_00876_b200 import binding as dl
    B, cap = len(lens), (max(lens) + 63) // 64 * 64
    cfg = wl.CONFIGS[2]
    q = wl.host_normal(cfg, wl.S_Q, (B, H, cap, D), dtype=dtype)
    k = wl.host_normal(cfg, wl.S_K, (B, H, cap, D), dtype=dtype)
    v = wl.host_normal(cfg, wl.S_V, (B, H, cap, D), dtype=dtype)
    if amp != 1.0:                               # power of two: stays exactly representable
        q, k = q * amp, k * amp
    scale = 1 / np.sqrt(D)
    n_max = max(lens)
    for impl in (1, 2):                          # CUDA cores; tensor cores
        ctx = _ctx(dtype, H, D, B=B, cap=cap)
        ctx.set_option(dl.DL_OPT_PREFILL_ATTN_IMPL, impl)
        out = torch.full((B, n_max, H, D), 7.0, dtype=wl.torch_dtype(dtype), device=DEV)
        qd, kd, vd = wl.to_torch(q, dtype, DEV), wl.to_torch(k, dtype, DEV), wl.to_torch(v, dtype, DEV)
        for b in range(B):                     # rows past the length are unspecified: make them hostile
            qd[b, :, lens[b]:] = float("nan")
            kd[b, :, lens[b]:] = float("nan")
            vd[b, :, lens[b]:] = float("nan")
        try:
            ctx.sparse_attn_prefill(qd, kd, vd, torch.tensor(lens, dtype=torch.int32, device=DEV), n_max, scale, out)
        except dl.DlError as e:
            assert impl >= 2 and e.code == dl.DL_ERR_UNSUPPORTED and not (dtype == "bf16" and D == 128)
            continue
        assert ctx.device_status()[0] == 0
        got = wl.from_torch(out)
        for b in range(B):
            n = lens[b]
            ref = np.stack([orc.attention_prefill_compact(q[b, h], k[b, h], v[b, h], n, scale) for h in range(H)], 1)
            pc.check_att(got[b, :n], ref, f"prefill impl {impl} seq {b} (n={n})")
            assert np.all(got[b, n:] == 7.0)                  # rows past the length are not written


@pytest.mark.parametrize("dtype,H,D,lens", [("f32", 8, 64, [68]), ("bf16", 4, 128, [208, 1, 130, 64]),
                                             ("bf16", 2, 128, [832, 300, 129, 128, 127, 65, 0]),
                                             ("bf16", 2, 64, [33, 100]), ("f32", 2, 128, [40, 7])])
def test_prefill_attention(dtype, H, D, lens):
    _prefill_case(dtype, H, D, lens)


def test_prefill_attention_tile_pair_boundaries():
    """Lengths on and around the 128-row query tiles, the 256-row tile pairs and the 16-key steps of the
    tensor-core kernel (a pair whose earlier tile is missing, clipped or full; last key tiles of 1..16 keys)."""
    _prefill_case("bf16", 2, 128, [256, 257, 255, 272, 240, 384, 385, 383])
    _prefill_case("bf16", 1, 128, [513, 512, 511, 16, 17, 15, 144, 145, 2])
    _prefill_case("bf16", 3, 128, [640])


def test_prefill_attention_top_rows_of_a_sequence():
    """Lengths that leave a top tile of 1..16 rows: alone in its pair (n = 256 m + r), beside a full later tile
    (n = 256 m + 128 + r), as the whole sequence, with r not a multiple of 16; those rows take a path of their own
    in the tensor-core kernel.  17 rows are the first length that does not."""
    _prefill_case("bf16", 2, 128, [261, 140, 400, 9, 16, 528, 272, 17])
    _prefill_case("bf16", 1, 128, [144, 133, 769, 3])


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_prefill_attention_random_ragged_batches(seed):
    """Many sequences of random lengths in one call (empty ones, lengths that leave a lane without a tile, top tiles of
    1..16 rows, several waves of items per CTA): the tensor-core kernel against the CUDA-core one, which the oracle
    checks in the cases above.  Rows past a sequence's length must stay untouched."""
    from paper_2412_00876_b200 import binding as dl
    rng = np.random.default_rng(100 + seed)
    B, H, D = 40, 8, 128
    lens = [int(v) for v in rng.integers(0, 900, B)]
    lens[3], lens[7], lens[11] = 0, 16, 128 + 16
    cap = (max(lens) + 63) // 64 * 64
    n_max = max(lens)
    cfg = wl.CONFIGS[5]
    mk = lambda s: wl.device_normal(cfg, s, (B, H, cap, D), DEV, sub=seed)
    q, k, v = mk(wl.S_Q), mk(wl.S_K), mk(wl.S_V)
    ln = torch.tensor(lens, dtype=torch.int32, device=DEV)
    outs = {}
    for impl in (2, 1):
        ctx = _ctx("bf16", H, D, B=B, cap=cap)
        ctx.set_option(dl.DL_OPT_PREFILL_ATTN_IMPL, impl)
        out = torch.full((B, n_max, H, D), 7.0, dtype=torch.bfloat16, device=DEV)
        ctx.sparse_attn_prefill(q, k, v, ln, n_max, 1 / np.sqrt(D), out)
        torch.cuda.synchronize()
        assert ctx.device_status()[0] == 0
        outs[impl] = wl.from_torch(out)
    for b in range(B):
        n = lens[b]
        assert np.all(outs[2][b, n:] == 7.0), b
        if n:
            mx, rl = pc.att_errors(outs[2][b, :n], outs[1][b, :n])
            assert mx <= pc.ATT_MAXABS and rl <= pc.ATT_RELL2, (b, n, mx, rl)


def test_prefill_attention_large_scores():
    """Scores whose row maximum keeps growing by far more than 2^8 from one key tile to the next: the
    tensor-core kernel has to rescale its accumulator and redo tiles (its rare path)."""
    _prefill_case("bf16", 2, 128, [600, 300, 129], amp=4.0)


def test_prefill_attention_large_grid_is_reproducible():
    """Several waves of work items per CTA: the tensor-core kernel must
    give the same bits every time and agree with the CUDA-core kernel (which the oracle checks above)."""
    from paper_2412_00876_b200 import binding as dl
    B, H, D, cap, n = 8, 32, 128, 1024, 832
    cfg = wl.CONFIGS[5]
    mk = lambda s: wl.device_normal(cfg, s, (B, H, cap, D), DEV)
    q, k, v = mk(wl.S_Q), mk(wl.S_K), mk(wl.S_V)
    ln = torch.full((B,), n, dtype=torch.int32, device=DEV)
    scale = 1 / np.sqrt(D)
    outs = {}
    for impl in (2, 1):
        ctx = _ctx("bf16", H, D, B=B, cap=cap)
        ctx.set_option(dl.DL_OPT_PREFILL_ATTN_IMPL, impl)
        first = None
        for rep in range(6 if impl != 1 else 1):
            out = torch.zeros(B, n, H, D, dtype=torch.bfloat16, device=DEV)
            ctx.sparse_attn_prefill(q, k, v, ln, n, scale, out)
            torch.cuda.synchronize()
            if first is None:
                first = out
            else:
                assert torch.equal(first.view(torch.int16), out.view(torch.int16)), f"run {rep} differs"
        outs[impl] = wl.from_torch(first)
        assert ctx.device_status()[0] == 0
    for impl in (2,):
        mx, rl = pc.att_errors(outs[impl], outs[1])
        assert mx <= pc.ATT_MAXABS and rl <= pc.ATT_RELL2, (impl, mx, rl)
