"""ctypes binding of libdl_sparse.so: same names as include/dl.h, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams are torch's); every step of the
path runs in the library's kernels.  There is no fallback: if the library has not been
built the import of this module's `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DL_SPARSE_CHECKED=1 in the environment selects the checked twin (stores through computed indices are compared with
# their buffers first; see include/dl.h)
LIB_PATH = os.path.join(_HERE, "libdl_sparse_checked.so" if os.environ.get("DL_SPARSE_CHECKED") == "1"
                        else "libdl_sparse.so")

DL_F32, DL_BF16 = 0, 1
DL_OK = 0
DL_ERR_INVALID_ARG, DL_ERR_ALIGNMENT, DL_ERR_UNSUPPORTED, DL_ERR_WORKSPACE = -1, -2, -3, -4
DL_ERR_CUDA, DL_ERR_CAPACITY, DL_ERR_TIMEOUT, DL_WARN_NAN = -5, -6, -7, 1
DL_ERR_BOUNDS = -8
DL_OPT_PREDICTOR_IMPL, DL_OPT_PREFILL_ATTN_IMPL, DL_OPT_DECODE_CHUNK, DL_OPT_DECODE_IMPL = 1, 2, 3, 4
DL_OPT_COMPACT_IMPL = 5

EXPORTS = [
    "dl_create", "dl_destroy", "dl_workspace_bytes", "dl_set_workspace", "dl_set_option",
    "dl_device_status", "dl_status_str", "dl_last_cuda_error", "dl_predictor_scores",
    "dl_topk_from_scores", "dl_prefill_select", "dl_compact_kv", "dl_sparse_attn_prefill",
    "dl_sparse_attn_decode", "dl_decode_keep", "dl_commit_len", "dl_decode_step", "dl_decode_step_host",
    "dl_sparse_attn_decode_static", "dl_sparse_attn_decode_layers", "dl_decode_nocache_select",
    "dl_decode_steps_host", "dl_compact_kv_host", "dl_selftest_wait_timeout", "dl_compact_kv_layers",
    "dl_predictor2_scratch_bytes", "dl_predictor2_values", "dl_prefill_select2", "dl_decode_keep2",
    "dl_decode_step_stack", "dl_quantize_kv_fp8", "dl_sparse_attn_decode_fp8", "dl_build_is_checked",
    "dl_selftest_bounds", "dl_sparse_attn_decode_fp8_layers",
]


class ModelDesc(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("pred_hidden", C.c_int32), ("dtype", C.c_int32)]


class LinearDesc(C.Structure):
    _fields_ = [("w", C.c_void_p), ("b", C.c_void_p)]


class VitBlockDesc(C.Structure):
    _fields_ = [("ln1_g", C.c_void_p), ("ln1_b", C.c_void_p), ("qkv", LinearDesc), ("proj", LinearDesc),
                ("ln2_g", C.c_void_p), ("ln2_b", C.c_void_p), ("fc1", LinearDesc), ("fc2", LinearDesc)]


class LayerStackDesc(C.Structure):
    _fields_ = [("L", C.c_int32), ("l_dense", C.c_int32), ("k_caches", C.POINTER(C.c_void_p)),
                ("v_caches", C.POINTER(C.c_void_p)), ("cap_dense", C.c_int32), ("cap", C.c_int32),
                ("len_dense", C.c_void_p), ("cache_len", C.c_void_p)]


class Predictor2Desc(C.Structure):
    _fields_ = [("inp", LinearDesc), ("n_blocks", C.c_int32), ("blocks", C.POINTER(VitBlockDesc)),
                ("h1", LinearDesc), ("h2", LinearDesc), ("w3", C.c_void_p), ("b3", C.c_void_p)]


class PredictorDesc(C.Structure):
    _fields_ = [("w1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p), ("b2", C.c_float)]


class Predictor2:
    """Device tensors of a predictor in the paper's architecture and the descriptor that points at them.
    `params` is the dictionary layout of workloads.make_predictor_paper with torch CUDA tensors as values
    (matrices bf16, vectors float32); the tensors are kept alive here."""

    def __init__(self, params: dict):
        self.params = params
        lin = lambda w, b: LinearDesc(w.data_ptr(), b.data_ptr())
        blocks = params["blocks"]
        self._blocks = (VitBlockDesc * max(len(blocks), 1))()
        for i, k in enumerate(blocks):
            self._blocks[i] = VitBlockDesc(k["ln1_g"].data_ptr(), k["ln1_b"].data_ptr(), lin(k["w_qkv"], k["b_qkv"]),
                                           lin(k["w_o"], k["b_o"]), k["ln2_g"].data_ptr(), k["ln2_b"].data_ptr(),
                                           lin(k["w_fc1"], k["b_fc1"]), lin(k["w_fc2"], k["b_fc2"]))
        h = params["head"]
        self.desc = Predictor2Desc(lin(params["w_in"], params["b_in"]), len(blocks),
                                   C.cast(self._blocks, C.POINTER(VitBlockDesc)), lin(h["w1"], h["b1"]),
                                   lin(h["w2"], h["b2"]), h["w3"].data_ptr(), h["b3"].data_ptr())


_lib = None


def lib() -> C.CDLL:
    """Opens the CUDA library (once).  Raises if it is missing: build it with
    `python -m paper_2412_00876_b200.build`."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2412_00876_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
        P = C.POINTER(PredictorDesc)
        sig = {
            "dl_create": (i32, [C.POINTER(vp), i32, C.POINTER(ModelDesc)]),
            "dl_destroy": (i32, [vp]),
            "dl_workspace_bytes": (i64, [vp, i32, i32, i32]),
            "dl_set_workspace": (i32, [vp, vp, i64, i32, i32, i32, vp]),
            "dl_set_option": (i32, [vp, i32, i32]),
            "dl_device_status": (i32, [vp, vp, C.POINTER(i32), C.POINTER(i64)]),
            "dl_status_str": (C.c_char_p, [i32]),
            "dl_last_cuda_error": (C.c_char_p, [vp]),
            "dl_predictor_scores": (i32, [vp, P, vp, i32, vp, vp]),
            "dl_topk_from_scores": (i32, [vp, vp, vp, vp, i32, i32, vp, i32, vp, vp]),
            "dl_prefill_select": (i32, [vp, P, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp]),
            "dl_compact_kv": (i32, [vp, vp, vp, vp, i32, vp, i32, i32, vp, vp, i32, vp, i32, vp]),
            "dl_compact_kv_host": (i32, [vp, vp, vp, vp, i32, vp, i32, i32, vp, vp, i32, vp, i32, vp]),
            "dl_compact_kv_layers": (i32, [vp, i32, C.POINTER(vp), C.POINTER(vp), vp, i32, vp, i32, i32, i32, vp, i32, vp]),
            "dl_sparse_attn_prefill": (i32, [vp, vp, vp, vp, vp, i32, i32, i32, f32, vp, vp]),
            "dl_sparse_attn_decode": (i32, [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp, vp]),
            "dl_sparse_attn_decode_static": (i32, [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp, vp]),
            "dl_sparse_attn_decode_layers": (i32, [vp, i32, vp, vp, vp, C.POINTER(vp), C.POINTER(vp), vp, vp, i32, i32,
                                                  f32, vp, vp]),
            "dl_decode_keep": (i32, [vp, P, vp, i32, f32, vp, vp, vp]),
            "dl_selftest_wait_timeout": (i32, [vp, i32, vp]),
            "dl_predictor2_scratch_bytes": (i64, [vp, i64]),
            "dl_predictor2_values": (i32, [vp, C.POINTER(Predictor2Desc), vp, vp, i32, i32, vp, i64, vp, vp, vp, vp]),
            "dl_prefill_select2": (i32, [vp, C.POINTER(Predictor2Desc), vp, vp, vp, i32, i32, vp, i64, vp, vp, vp, i32,
                                         vp, vp]),
            "dl_decode_keep2": (i32, [vp, C.POINTER(Predictor2Desc), vp, i32, vp, i64, vp, vp, vp]),
            "dl_decode_nocache_select": (i32, [vp, P, vp, vp, i32, i32, f32, vp, vp, vp]),
            "dl_commit_len": (i32, [vp, vp, i32, i32, vp, vp]),
            "dl_decode_step": (i32, [vp, P, vp, i32, f32, vp, vp, i32, vp, vp, vp, C.POINTER(vp),
                                     C.POINTER(vp), i32, vp, f32, vp, vp]),
            "dl_decode_step_stack": (i32, [vp, P, vp, i32, f32, vp, vp, C.POINTER(LayerStackDesc), vp, vp, vp, f32,
                                           vp, vp]),
            "dl_sparse_attn_decode_fp8_layers": (i32, [vp, i32, vp, vp, vp, C.POINTER(vp), C.POINTER(vp), vp, vp, vp, vp,
                                                       i32, i32, f32, vp, i32, vp]),
            "dl_build_is_checked": (i32, []),
            "dl_selftest_bounds": (i32, [vp, vp]),
            "dl_quantize_kv_fp8": (i32, [vp, vp, vp, vp, i32, i32, vp, vp]),
            "dl_sparse_attn_decode_fp8": (i32, [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp, vp]),
            "dl_decode_step_host": (i32, [vp, P, vp, i32, f32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                          vp, vp, C.POINTER(vp), C.POINTER(vp), i32, vp, f32, vp]),
            "dl_decode_steps_host": (i32, [vp, P, i32, i32, f32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                           C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, vp, vp, vp, vp, vp, vp,
                                           C.POINTER(vp), C.POINTER(vp), i32, vp, f32, vp]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class DlError(RuntimeError):
    def __init__(self, code: int, where: str, extra: str = ""):
        self.code = code
        msg = lib().dl_status_str(code).decode()
        super().__init__(f"{where}: {msg} ({code}){' - ' + extra if extra else ''}")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        if not t.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return t.data_ptr()
    return int(t)


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


class Predictor:
    """Device copy of one predictor's weights (see dl_predictor in dl.h)."""

    def __init__(self, w1: torch.Tensor, b1: torch.Tensor, w2: torch.Tensor, b2: float):
        assert b1.dtype == torch.float32 and w2.dtype == torch.float32
        self.w1, self.b1, self.w2, self.b2 = w1.contiguous(), b1.contiguous(), w2.contiguous(), float(b2)
        self.desc = PredictorDesc(self.w1.data_ptr(), self.b1.data_ptr(), self.w2.data_ptr(), self.b2)


class Context:
    """Owns a dl_ctx and the torch tensor that serves as its workspace."""

    def __init__(self, hidden: int, n_heads: int, head_dim: int, pred_hidden: int, dtype: torch.dtype,
                 device: int = 0, max_batch: int = 1, max_rows: int = 0, cap: int = 64):
        self._h = C.c_void_p()
        self.dtype = dtype
        self.device = torch.device("cuda", device)
        self.H, self.D, self.hidden = n_heads, head_dim, hidden
        d = ModelDesc(hidden, n_heads, head_dim, pred_hidden, DL_F32 if dtype == torch.float32 else DL_BF16)
        st = lib().dl_create(C.byref(self._h), device, C.byref(d))
        if st != DL_OK:
            raise DlError(st, "dl_create")
        self._ws = None
        self.set_workspace(max_batch, max(max_rows, max_batch), cap)

    def close(self):
        if self._h:
            lib().dl_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, where: str):
        if st != DL_OK:
            extra = lib().dl_last_cuda_error(self._h).decode() if st == DL_ERR_CUDA else ""
            raise DlError(st, where, extra)

    # ---- context calls
    def set_workspace(self, max_batch: int, max_rows: int, cap: int, stream=None):
        n = lib().dl_workspace_bytes(self._h, max_batch, max_rows, cap)
        if n < 0:
            raise DlError(int(n), "dl_workspace_bytes")
        self._ws = torch.empty(int(n) + 256, dtype=torch.uint8, device=self.device)
        base = (self._ws.data_ptr() + 255) // 256 * 256
        self._check(lib().dl_set_workspace(self._h, base, n, max_batch, max_rows, cap, _stream(stream)),
                    "dl_set_workspace")
        self.max_batch, self.max_rows, self.cap = max_batch, max_rows, cap

    def set_option(self, option: int, value: int):
        self._check(lib().dl_set_option(self._h, option, value), "dl_set_option")

    def device_status(self, stream=None):
        code, detail = C.c_int32(0), C.c_int64(0)
        self._check(lib().dl_device_status(self._h, _stream(stream), C.byref(code), C.byref(detail)),
                    "dl_device_status")
        return code.value, detail.value

    # ---- the path
    def predictor_scores(self, p: Predictor, x, score_out, stream=None):
        rows = x.numel() // self.hidden
        self._check(lib().dl_predictor_scores(self._h, C.byref(p.desc), _ptr(x), rows, _ptr(score_out),
                                              _stream(stream)), "dl_predictor_scores")

    def topk_from_scores(self, score, n_vis, k, kept_idx_out, keep_out, stream=None):
        B, n_max = score.shape
        k_max = 0 if kept_idx_out is None else kept_idx_out.shape[1]
        self._check(lib().dl_topk_from_scores(self._h, _ptr(score), _ptr(n_vis), _ptr(k), B, n_max,
                                              _ptr(kept_idx_out), k_max, _ptr(keep_out), _stream(stream)),
                    "dl_topk_from_scores")

    def prefill_select(self, p: Predictor, x_vis, n_vis, k, score_out, kept_idx_out, keep_out, stream=None):
        B, n_max = x_vis.shape[0], x_vis.shape[1]
        k_max = 0 if kept_idx_out is None else kept_idx_out.shape[1]
        self._check(lib().dl_prefill_select(self._h, C.byref(p.desc), _ptr(x_vis), _ptr(n_vis), _ptr(k), B,
                                            n_max, _ptr(score_out), _ptr(kept_idx_out), k_max, _ptr(keep_out),
                                            _stream(stream)), "dl_prefill_select")

    def compact_kv(self, k_src, v_src, keep, t_src, k_cache, v_cache, cache_len, commit=True, stream=None):
        B, T = k_src.shape[0], k_src.shape[1]
        cap = k_cache.shape[2]
        keep_cols = 0 if keep is None else keep.shape[1]
        self._check(lib().dl_compact_kv(self._h, _ptr(k_src), _ptr(v_src), _ptr(keep), keep_cols, _ptr(t_src), B, T,
                                        _ptr(k_cache), _ptr(v_cache), cap, _ptr(cache_len), int(bool(commit)),
                                        _stream(stream)), "dl_compact_kv")

    def compact_kv_layers(self, srcs, caches, keep, t_src, cache_len, commit=True, stream=None):
        """dl_compact_kv_layers: len(srcs) tensors (K, V, Q ... of any number of layers) under one decision."""
        n = len(srcs)
        B, T = srcs[0].shape[0], srcs[0].shape[1]
        cap = caches[0].shape[2]
        keep_cols = 0 if keep is None else keep.shape[1]
        sp, cp = self.pointer_array(srcs), self.pointer_array(caches)
        self._check(lib().dl_compact_kv_layers(self._h, n, sp, cp, _ptr(keep), keep_cols, _ptr(t_src), B, T, cap,
                                               _ptr(cache_len), int(bool(commit)), _stream(stream)),
                    "dl_compact_kv_layers")

    def compact_kv_host(self, k_src_host, v_src_host, keep, t_src, k_cache, v_cache, cache_len, commit=True,
                        stream=None):
        """dl_compact_kv with the source rows in pinned host tensors: the kernel fetches the kept rows itself."""
        B, T = k_src_host.shape[0], k_src_host.shape[1]
        cap = k_cache.shape[2]
        keep_cols = 0 if keep is None else keep.shape[1]
        self._check(lib().dl_compact_kv_host(self._h, _ptr(k_src_host), _ptr(v_src_host), _ptr(keep), keep_cols,
                                             _ptr(t_src), B, T, _ptr(k_cache), _ptr(v_cache), cap, _ptr(cache_len),
                                             int(bool(commit)), _stream(stream)), "dl_compact_kv_host")

    def sparse_attn_prefill(self, q, k_cache, v_cache, cache_len, n_max, scale, out, stream=None):
        B, cap = k_cache.shape[0], k_cache.shape[2]
        self._check(lib().dl_sparse_attn_prefill(self._h, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(cache_len),
                                                 B, cap, n_max, float(scale), _ptr(out), _stream(stream)),
                    "dl_sparse_attn_prefill")

    def sparse_attn_decode(self, q_t, k_t, v_t, k_cache, v_cache, cache_len, keep, scale, out, stream=None):
        B, cap = k_cache.shape[0], k_cache.shape[2]
        self._check(lib().dl_sparse_attn_decode(self._h, _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(k_cache),
                                                _ptr(v_cache), _ptr(cache_len), _ptr(keep), B, cap, float(scale),
                                                _ptr(out), _stream(stream)), "dl_sparse_attn_decode")

    def selftest_bounds(self, stream=None):
        """Checked build: one store a word past a buffer's end, which must be skipped and recorded."""
        return lib().dl_selftest_bounds(self._h, _stream(stream))

    def quantize_kv_fp8(self, src, cache_len, scale, dst, stream=None):
        """Extension (not in the paper): rows of a bf16 cache as E4M3 bytes under per-head scales."""
        B, cap = src.shape[0], src.shape[2]
        self._check(lib().dl_quantize_kv_fp8(self._h, _ptr(src), _ptr(cache_len), _ptr(scale), B, cap, _ptr(dst),
                                             _stream(stream)), "dl_quantize_kv_fp8")

    def sparse_attn_decode_fp8(self, q_t, k_t, v_t, k_cache, v_cache, k_scale, v_scale, cache_len, keep, scale, out,
                               stream=None):
        B, cap = k_cache.shape[0], k_cache.shape[2]
        self._check(lib().dl_sparse_attn_decode_fp8(self._h, _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(k_cache),
                                                    _ptr(v_cache), _ptr(k_scale), _ptr(v_scale), _ptr(cache_len),
                                                    _ptr(keep), B, cap, float(scale), _ptr(out), _stream(stream)),
                    "dl_sparse_attn_decode_fp8")

    def sparse_attn_decode_fp8_layers(self, q_t, k_t, v_t, k_caches, v_caches, k_scales, v_scales, cache_len, keep,
                                      scale, out, commit=False, stream=None):
        """k_caches / v_caches: lists of the L layers' byte caches; k_scales / v_scales [L][H]."""
        L, B, cap = len(k_caches), k_caches[0].shape[0], k_caches[0].shape[2]
        kp, vp_ = self.pointer_array(k_caches), self.pointer_array(v_caches)
        self._check(lib().dl_sparse_attn_decode_fp8_layers(
            self._h, L, _ptr(q_t), _ptr(k_t), _ptr(v_t), kp, vp_, _ptr(k_scales), _ptr(v_scales), _ptr(cache_len),
            _ptr(keep), B, cap, float(scale), _ptr(out), int(bool(commit)), _stream(stream)),
            "dl_sparse_attn_decode_fp8_layers")

    def sparse_attn_decode_static(self, q_t, k_t, v_t, k_cache, v_cache, cache_len, keep, scale, out, stream=None):
        """dl_sparse_attn_decode for callers that may not allocate device memory: the kernel's scratch
        is the library's built-in array (see dl.h for its size limit and the sharing rules)."""
        B, cap = k_cache.shape[0], k_cache.shape[2]
        self._check(lib().dl_sparse_attn_decode_static(self._h, _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(k_cache),
                                                       _ptr(v_cache), _ptr(cache_len), _ptr(keep), B, cap,
                                                       float(scale), _ptr(out), _stream(stream)),
                    "dl_sparse_attn_decode_static")

    def sparse_attn_decode_layers(self, q_t, k_t, v_t, k_ptrs, v_ptrs, L, cap, cache_len, keep, scale, out,
                                  stream=None):
        B = cache_len.shape[0]
        self._check(lib().dl_sparse_attn_decode_layers(self._h, L, _ptr(q_t), _ptr(k_t), _ptr(v_t), k_ptrs, v_ptrs,
                                                       _ptr(cache_len), _ptr(keep), B, cap, float(scale), _ptr(out),
                                                       _stream(stream)), "dl_sparse_attn_decode_layers")

    def decode_keep(self, p: Predictor | None, x_t, logit_inout, keep_out, threshold=0.0, stream=None):
        B = logit_inout.shape[0]
        pd = C.byref(p.desc) if p is not None else None
        self._check(lib().dl_decode_keep(self._h, pd, _ptr(x_t), B, float(threshold), _ptr(logit_inout),
                                         _ptr(keep_out), _stream(stream)), "dl_decode_keep")

    def decode_nocache_select(self, p: Predictor | None, x_gen, n_gen, logit_inout, keep_out, threshold=0.0,
                              stream=None):
        B, n_max = logit_inout.shape
        pd = C.byref(p.desc) if p is not None else None
        self._check(lib().dl_decode_nocache_select(self._h, pd, _ptr(x_gen), _ptr(n_gen), B, n_max, float(threshold),
                                                   _ptr(logit_inout), _ptr(keep_out), _stream(stream)),
                    "dl_decode_nocache_select")

    def commit_len(self, keep, cache_len, cap, stream=None):
        self._check(lib().dl_commit_len(self._h, _ptr(keep), keep.shape[0], cap, _ptr(cache_len),
                                        _stream(stream)), "dl_commit_len")

    # ---- the paper's own predictors
    def predictor2_scratch(self, rows: int) -> torch.Tensor:
        """Scratch tensor of the size dl_predictor2_values wants for `rows` rows."""
        n = lib().dl_predictor2_scratch_bytes(self._h, int(rows))
        if n < 0:
            raise DlError(int(n), "dl_predictor2_scratch_bytes")
        return torch.empty(max(int(n), 256), dtype=torch.uint8, device=self.device)

    def predictor2_values(self, p: "Predictor2", x, n_vis, scratch, d_out=None, score_out=None, keep_out=None, stream=None):
        B, n_max = x.shape[0], x.shape[1]
        self._check(lib().dl_predictor2_values(self._h, C.byref(p.desc), _ptr(x), _ptr(n_vis), B, n_max, _ptr(scratch),
                                               scratch.numel(), _ptr(d_out), _ptr(score_out), _ptr(keep_out),
                                               _stream(stream)), "dl_predictor2_values")

    def prefill_select2(self, p: "Predictor2", x_vis, n_vis, k, scratch, d_out, score_out, kept_idx_out, keep_out,
                        stream=None):
        B, n_max = x_vis.shape[0], x_vis.shape[1]
        self._check(lib().dl_prefill_select2(self._h, C.byref(p.desc), _ptr(x_vis), _ptr(n_vis), _ptr(k), B, n_max,
                                             _ptr(scratch), scratch.numel(), _ptr(d_out), _ptr(score_out),
                                             _ptr(kept_idx_out), kept_idx_out.shape[1], _ptr(keep_out), _stream(stream)),
                    "dl_prefill_select2")

    def decode_keep2(self, p: "Predictor2", x_t, scratch, d_out, keep_out, stream=None):
        self._check(lib().dl_decode_keep2(self._h, C.byref(p.desc), _ptr(x_t), x_t.shape[0], _ptr(scratch),
                                          scratch.numel(), _ptr(d_out), _ptr(keep_out), _stream(stream)),
                    "dl_decode_keep2")

    def selftest_wait_timeout(self, polls: int = 64, stream=None):
        self._check(lib().dl_selftest_wait_timeout(self._h, int(polls), _stream(stream)), "dl_selftest_wait_timeout")

    @staticmethod
    def pointer_array(tensors):
        arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
        return arr

    def decode_step(self, p: Predictor | None, x_t, logit_inout, keep_out, q_t, k_t, v_t, k_ptrs, v_ptrs, L,
                    cap, cache_len, scale, out, threshold=0.0, stream=None):
        B = logit_inout.shape[0]
        pd = C.byref(p.desc) if p is not None else None
        self._check(lib().dl_decode_step(self._h, pd, _ptr(x_t), B, float(threshold), _ptr(logit_inout),
                                         _ptr(keep_out), L, _ptr(q_t), _ptr(k_t), _ptr(v_t), k_ptrs, v_ptrs, cap,
                                         _ptr(cache_len), float(scale), _ptr(out), _stream(stream)),
                    "dl_decode_step")

    def decode_step_stack(self, p: Predictor | None, x_t, logit_inout, keep_out, k_caches, v_caches, l_dense,
                          cap_dense, cap, len_dense, cache_len, q_t, k_t, v_t, scale, out, threshold=0.0,
                          stream=None):
        """One decode step over a stack whose first l_dense layers keep every token (k_caches / v_caches: lists of
        the L layers' cache tensors)."""
        B, L = logit_inout.shape[0], len(k_caches)
        kp = (C.c_void_p * max(L, 1))(*[t.data_ptr() for t in k_caches])
        vp_ = (C.c_void_p * max(L, 1))(*[t.data_ptr() for t in v_caches])
        st = LayerStackDesc(L, l_dense, kp, vp_, cap_dense, cap, _ptr(len_dense), _ptr(cache_len))
        pd = C.byref(p.desc) if p is not None else None
        self._check(lib().dl_decode_step_stack(self._h, pd, _ptr(x_t), B, float(threshold), _ptr(logit_inout),
                                               _ptr(keep_out), C.byref(st), _ptr(q_t), _ptr(k_t), _ptr(v_t),
                                               float(scale), _ptr(out), _stream(stream)), "dl_decode_step_stack")

    def decode_steps_host(self, p: Predictor, x_hosts, q_hosts, k_hosts, v_hosts, out_hosts, keep_hosts, stage_x,
                          stage_q, stage_k, stage_v, stage_out, logit_dev, keep_dev, k_ptrs, v_ptrs, L, cap,
                          cache_len, scale, threshold=0.0, stream=None):
        """len(x_hosts) decode steps fed from (pinned) host tensors, copies pipelined against the compute;
        the staging tensors hold two sets each (leading dimension 2)."""
        n = len(x_hosts)
        B = logit_dev.shape[-1]
        arr = lambda ts: (C.c_void_p * n)(*[(t.data_ptr() if t is not None else None) for t in ts])
        keep_arr = arr(keep_hosts) if keep_hosts is not None else None
        self._check(lib().dl_decode_steps_host(
            self._h, C.byref(p.desc), n, B, float(threshold), L, arr(x_hosts), arr(q_hosts), arr(k_hosts),
            arr(v_hosts), arr(out_hosts), keep_arr, _ptr(stage_x), _ptr(stage_q), _ptr(stage_k), _ptr(stage_v),
            _ptr(stage_out), _ptr(logit_dev), _ptr(keep_dev), k_ptrs, v_ptrs, cap, _ptr(cache_len), float(scale),
            _stream(stream)), "dl_decode_steps_host")

    def decode_step_host(self, p: Predictor, x_host, q_host, k_host, v_host, out_host, keep_host, stage_x,
                         stage_q, stage_k, stage_v, stage_out, logit_dev, keep_dev, k_ptrs, v_ptrs, L, cap,
                         cache_len, scale, threshold=0.0, stream=None):
        B = logit_dev.shape[0]
        self._check(lib().dl_decode_step_host(
            self._h, C.byref(p.desc), _ptr(x_host), B, float(threshold), L, _ptr(q_host), _ptr(k_host),
            _ptr(v_host), _ptr(out_host), _ptr(keep_host), _ptr(stage_x), _ptr(stage_q), _ptr(stage_k),
            _ptr(stage_v), _ptr(stage_out), _ptr(logit_dev), _ptr(keep_dev), k_ptrs, v_ptrs, cap,
            _ptr(cache_len), float(scale), _stream(stream)), "dl_decode_step_host")
