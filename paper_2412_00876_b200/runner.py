"""Drives one batch of requests through the whole path with the library's calls:
prefill select -> compaction of every layer's K/V (and Q) -> prefill attention per layer ->
N_OT decode steps (keep decision, per-layer attention with fused append, length commit).

This is the loop a serving engine would run around the projections and FFNs it owns; here the
projected activations are synthetic tensors that already sit in device memory (or, for the
host-fed variant, in pinned host memory).  Only argument marshalling happens in Python.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as dl
from . import workloads as wl


class BatchRunner:
    """Buffers and call sequence for one workload configuration on one GPU."""

    def __init__(self, cfg: wl.Config, device: int = 0, rank: int = 0, src_pool: int = 4, step_pool: int = 8,
                 host_fed: bool = False, options: dict | None = None, use_graphs: bool = False):
        self.cfg, self.dev, self.rank = cfg, torch.device("cuda", device), rank
        B, L, H, D = cfg.B, cfg.n_layers, cfg.n_heads, cfg.head_dim
        self.T = cfg.n_vis + cfg.n_text
        self.cap = cfg.cap
        self.scale = 1.0 / float(np.sqrt(D))
        tdt = wl.torch_dtype(cfg.dtype)
        self.ctx = dl.Context(cfg.hidden, H, D, cfg.pred_hidden, tdt, device, max_batch=B,
                              max_rows=B * cfg.n_vis, cap=self.cap)
        for o, v in (options or {}).items():
            self.ctx.set_option(o, v)
        dev = self.dev

        def pred(which):
            p = wl.make_predictor(cfg, which)
            return p, dl.Predictor(wl.to_torch(p.w1, cfg.dtype, dev), torch.from_numpy(p.b1).to(dev),
                                   torch.from_numpy(p.w2).to(dev), p.b2)

        self.p_img_host, self.p_img = pred("img")
        self.p_txt_host, self.p_txt = pred("txt")
        sub = 1000 * rank
        # ---- prefill inputs: pools larger than L2, cycled over the layers
        self.src_pool = min(src_pool, L)
        self.step_pool = min(step_pool, max(cfg.n_gen, 1))
        self.x_vis = wl.device_normal(cfg, wl.S_X_VIS, (B, cfg.n_vis, cfg.hidden), dev, sub=sub)
        shape = (B, self.T, H, D)
        self.q_src = [wl.device_normal(cfg, wl.S_Q, shape, dev, sub=sub + i) for i in range(self.src_pool)]
        self.k_src = [wl.device_normal(cfg, wl.S_K, shape, dev, sub=sub + i) for i in range(self.src_pool)]
        self.v_src = [wl.device_normal(cfg, wl.S_V, shape, dev, sub=sub + i) for i in range(self.src_pool)]
        # ---- decode inputs
        P = self.step_pool
        self.x_dec = wl.device_normal(cfg, wl.S_X_TXT, (P, B, cfg.hidden), dev, sub=sub)
        self.q_dec = wl.device_normal(cfg, wl.S_DEC_Q, (P, L, B, H, D), dev, sub=sub)
        self.k_dec = wl.device_normal(cfg, wl.S_DEC_K, (P, L, B, H, D), dev, sub=sub)
        self.v_dec = wl.device_normal(cfg, wl.S_DEC_V, (P, L, B, H, D), dev, sub=sub)
        # ---- state and outputs
        i32 = dict(dtype=torch.int32, device=dev)
        self.k_cache = [torch.empty(B, H, self.cap, D, dtype=tdt, device=dev) for _ in range(L)]
        self.v_cache = [torch.empty(B, H, self.cap, D, dtype=tdt, device=dev) for _ in range(L)]
        self.q_cache = torch.empty(B, H, self.cap, D, dtype=tdt, device=dev)
        self.kp, self.vp = self.ctx.pointer_array(self.k_cache), self.ctx.pointer_array(self.v_cache)
        self.cache_len = torch.zeros(B, **i32)
        self.q_len = torch.zeros(B, **i32)
        self.n_vis = torch.full((B,), cfg.n_vis, **i32)
        self.k_arr = torch.full((B,), cfg.k_vis, **i32)
        self.t_src = torch.full((B,), self.T, **i32)
        self.score = torch.empty(B, cfg.n_vis, dtype=torch.float32, device=dev)
        self.kept_idx = torch.empty(B, cfg.k_vis, **i32)
        self.keep_vis = torch.empty(B, cfg.n_vis, dtype=torch.uint8, device=dev)
        self.prefill_out = torch.empty(B, cfg.n0, H, D, dtype=tdt, device=dev)
        self.logit = torch.empty(B, dtype=torch.float32, device=dev)
        self.keep_t = torch.empty(B, dtype=torch.uint8, device=dev)
        self.dec_out = torch.empty(L, B, H, D, dtype=tdt, device=dev)
        self.launches = 0
        # launches of dl_decode_step: predictor (+ keep test unless fused: bf16) + L attention (+ nothing: commit folded)
        self.step_launches = (1 if cfg.dtype == "bf16" else 2) + cfg.n_layers
        self.use_graphs = use_graphs
        self._graphs: dict = {}            # decode step captured once per input-pool slot
        self.host_fed = host_fed
        if host_fed:
            self._make_host_buffers()

    # ------------------------------------------------------------------ device-resident path
    def prefill(self):
        c, ctx, L = self.cfg, self.ctx, self.cfg.n_layers
        self.cache_len.zero_()
        ctx.prefill_select(self.p_img, self.x_vis, self.n_vis, self.k_arr, self.score, self.kept_idx, self.keep_vis)
        self.launches += 2
        # K and V of every layer under the one decision: one plan, one run of overlapped copy launches
        srcs, caches = [], []
        for l in range(L):
            i = l % self.src_pool
            srcs += [self.k_src[i], self.v_src[i]]
            caches += [self.k_cache[l], self.v_cache[l]]
        ctx.compact_kv_layers(srcs, caches, self.keep_vis, self.t_src, self.cache_len, commit=True)
        self.launches += 1 + L
        for l in range(L):
            i = l % self.src_pool
            ctx.compact_kv(self.q_src[i], None, self.keep_vis, self.t_src, self.q_cache, None, self.q_len, commit=False)
            ctx.sparse_attn_prefill(self.q_cache, self.k_cache[l], self.v_cache[l], self.cache_len, c.n0, self.scale,
                                    self.prefill_out)
        self.launches += 3 * L

    def decode_step(self, t: int):
        c, i = self.cfg, t % self.step_pool
        if self.use_graphs:
            # The step's launches depend on the step only through device memory (lengths, flags, the pool
            # slot's inputs), so one captured graph per pool slot replays any step.
            g = self._graphs.get(i)
            if g is None:
                saved = self.cache_len.clone()
                self._decode_step_eager(i)                     # warm run: attributes set, tensor maps cached
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    self._decode_step_eager(i)
                self.cache_len.copy_(saved)                    # undo the warm run's commit (its appended row
                self._graphs[i] = g                            # lies past the restored length)
            g.replay()
            self.launches += self.step_launches
            return
        self._decode_step_eager(i)
        self.launches += self.step_launches

    def _decode_step_eager(self, i: int):
        c = self.cfg
        self.ctx.decode_step(self.p_txt, self.x_dec[i], self.logit, self.keep_t, self.q_dec[i], self.k_dec[i],
                             self.v_dec[i], self.kp, self.vp, c.n_layers, self.cap, self.cache_len, self.scale,
                             self.dec_out)

    def decode_step_timed(self, t: int, events: list):
        """The same step issued as keep decision, layer stack, commit, with one event pair around the
        stack's L attention launches (issued exactly as dl_decode_step issues them)."""
        c, i, ctx = self.cfg, t % self.step_pool, self.ctx
        ctx.decode_keep(self.p_txt, self.x_dec[i], self.logit, self.keep_t)
        lens = self.cache_len.clone()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.sparse_attn_decode_layers(self.q_dec[i], self.k_dec[i], self.v_dec[i], self.kp, self.vp, c.n_layers,
                                      self.cap, self.cache_len, self.keep_t, self.scale, self.dec_out)
        e1.record()
        events.append((e0, e1, lens, c.n_layers))
        ctx.commit_len(self.keep_t, self.cache_len, self.cap)
        self.launches += self.step_launches + 1

    def run_batch(self, sample_every: int = 0, events: list | None = None):
        """One whole batch.  With `sample_every`, every sample_every-th decode step is issued call by
        call with events around its attention launches; the prefill and those steps sit inside an
        NVTX range ("dl_sample") so that a profiler can be told to look at them only."""
        nvtx = torch.cuda.nvtx
        if sample_every:
            nvtx.range_push("dl_sample")
        self.prefill()
        if sample_every:
            nvtx.range_pop()
        for t in range(self.cfg.n_gen):
            if sample_every and events is not None and t % sample_every == sample_every - 1:
                nvtx.range_push("dl_sample")
                self.decode_step_timed(t, events)
                nvtx.range_pop()
            else:
                self.decode_step(t)

    def decode_bytes(self, lens: torch.Tensor) -> int:
        """Algorithmic bytes of one decode-attention launch: every valid cached K and V row and the
        current token's row once, plus q and the output."""
        c = self.cfg
        rows = int(lens.sum().item()) + c.B
        return (2 * rows + 2 * c.B) * c.n_heads * c.head_dim * c.elt_bytes

    # ------------------------------------------------------------------ host-fed path
    def _make_host_buffers(self):
        def pin(t):
            return t.cpu().pin_memory()
        self.h_x_vis = pin(self.x_vis)
        self.h_q_src = [pin(t) for t in self.q_src]
        self.h_k_src = [pin(t) for t in self.k_src]
        self.h_v_src = [pin(t) for t in self.v_src]
        self.h_x_dec, self.h_q_dec = pin(self.x_dec), pin(self.q_dec)
        self.h_k_dec, self.h_v_dec = pin(self.k_dec), pin(self.v_dec)
        self.h_prefill_out = torch.empty_like(self.prefill_out, device="cpu").pin_memory()
        # the host-fed prefill copies a layer's output out on a side stream while the next layer runs: two device buffers
        self.prefill_out2 = [self.prefill_out, torch.empty_like(self.prefill_out)]
        self.out_stream = torch.cuda.Stream(device=self.prefill_out.device)
        self.out_done = [torch.cuda.Event(), torch.cuda.Event()]
        self.out_ready = [torch.cuda.Event(), torch.cuda.Event()]
        self.h_dec_out = torch.empty_like(self.dec_out, device="cpu").pin_memory()
        self.h_keep = torch.empty(self.cfg.B, dtype=torch.uint8).pin_memory()
        # two staging sets each: the pipelined host-fed decode copies step t+1 in while step t computes
        two = lambda t: torch.empty((2,) + tuple(t.shape), dtype=t.dtype, device=t.device)
        self.s_x = two(self.x_dec[0])
        self.s_q, self.s_k, self.s_v, self.s_out = (two(self.q_dec[0]) for _ in range(4))
        self.s_logit, self.s_keep = two(self.logit), two(self.keep_t)
        self.h_dec_out2 = [torch.empty_like(self.dec_out, device="cpu").pin_memory() for _ in range(2)]
        self.h_keep2 = [torch.empty(self.cfg.B, dtype=torch.uint8).pin_memory() for _ in range(2)]
        self.s_xvis = torch.empty_like(self.x_vis)

    def run_batch_host_fed(self):
        """Same batch with every input copied from pinned host memory inside the call sequence
        and every result copied back; returns (h2d_bytes, d2h_bytes)."""
        c, ctx, L = self.cfg, self.ctx, self.cfg.n_layers
        h2d = d2h = 0
        self.cache_len.zero_()
        self.s_xvis.copy_(self.h_x_vis, non_blocking=True)
        h2d += self.h_x_vis.numel() * self.h_x_vis.element_size()
        ctx.prefill_select(self.p_img, self.s_xvis, self.n_vis, self.k_arr, self.score, self.kept_idx, self.keep_vis)
        # the per-layer Q/K/V sources stay in pinned host memory: the compaction kernel fetches the kept rows
        # itself, so the dropped rows never cross the bus (bytes counted: the kept rows)
        row_bytes = c.n_heads * c.head_dim * c.elt_bytes
        kept_bytes = c.B * c.n0 * row_bytes
        for l in range(L):
            i = l % self.src_pool
            h2d += 2 * kept_bytes
            ctx.compact_kv_host(self.h_k_src[i], self.h_v_src[i], self.keep_vis, self.t_src, self.k_cache[l],
                                self.v_cache[l], self.cache_len, commit=(l == L - 1))
        for l in range(L):
            i = l % self.src_pool
            h2d += kept_bytes
            ctx.compact_kv_host(self.h_q_src[i], None, self.keep_vis, self.t_src, self.q_cache, None, self.q_len,
                                commit=False)
            buf = self.prefill_out2[l & 1]
            main = torch.cuda.current_stream()
            if l >= 2:
                main.wait_event(self.out_done[l & 1])          # the copy out of this buffer, two layers ago
            ctx.sparse_attn_prefill(self.q_cache, self.k_cache[l], self.v_cache[l], self.cache_len, c.n0, self.scale, buf)
            self.out_ready[l & 1].record(main)
            with torch.cuda.stream(self.out_stream):
                self.out_stream.wait_event(self.out_ready[l & 1])
                self.h_prefill_out.copy_(buf, non_blocking=True)
                self.out_done[l & 1].record(self.out_stream)
            d2h += buf.numel() * buf.element_size()
        torch.cuda.current_stream().wait_stream(self.out_stream)
        per_step_in = (self.s_x[0].numel() + 3 * self.s_q[0].numel()) * self.s_x.element_size()
        per_step_out = self.dec_out.numel() * self.dec_out.element_size() + c.B
        # the decode steps as one pipelined host-fed call per chunk of steps (results land in two host
        # buffers in turn: a consumer would read step t's while step t+1 computes)
        chunk = 256
        for t0 in range(0, c.n_gen, chunk):
            steps = range(t0, min(c.n_gen, t0 + chunk))
            pool = [t % self.step_pool for t in steps]
            ctx.decode_steps_host(self.p_txt, [self.h_x_dec[i] for i in pool], [self.h_q_dec[i] for i in pool],
                                  [self.h_k_dec[i] for i in pool], [self.h_v_dec[i] for i in pool],
                                  [self.h_dec_out2[t & 1] for t in steps], [self.h_keep2[t & 1] for t in steps],
                                  self.s_x, self.s_q, self.s_k, self.s_v, self.s_out, self.s_logit, self.s_keep,
                                  self.kp, self.vp, L, self.cap, self.cache_len, self.scale)
            h2d += per_step_in * len(steps)
            d2h += per_step_out * len(steps)
        return h2d, d2h

    def close(self):
        self.ctx.close()
