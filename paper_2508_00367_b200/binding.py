"""Thin ctypes binding of librs.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch supplies
device memory and the current stream.  There is no CPU or eager fallback: if
the shared library is missing, or a call returns an error code, a RuntimeError
is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librs.so")

RS_OK = 0
RS_F32, RS_BF16 = 0, 1
DIST = {"l2": 0, "l1": 1, "cos": 2}
SCORE_MODE = {"mlp": 0, "mlp_delta": 1, "attn": 2, "block": 3}
STATUS_NAMES = {0: "RS_OK", 1: "RS_ERR_INVALID_ARG", 2: "RS_ERR_UNSUPPORTED", 3: "RS_ERR_WORKSPACE",
                4: "RS_ERR_CUDA", 5: "RS_ERR_TIMEOUT"}

EXPORTS = ("rs_create", "rs_destroy", "rs_last_error", "rs_async_status", "rs_uses_tensor_cores",
           "rs_launch_count", "rs_attn_fwd", "rs_shift_score", "rs_topk_compact",
           "rs_block_workspace_bytes", "rs_block_fwd", "rs_timing_enable", "rs_timing_read",
           "rs_static_scratch_bytes", "rs_block_fwd_static", "rs_linear_fwd", "rs_vit_workspace_bytes", "rs_vit_fwd",
           "rs_vit_fwd_taps", "rs_linewise_compact", "rs_static_async_status", "rs_linear_uses_tensor_cores",
           "rs_block_uses_tensor_cores", "rs_attn_fwd_ragged", "rs_topk_compact_ragged", "rs_block_fwd_ragged", "rs_vit_fwd_ragged", "rs_prepare_ln1_fold", "rs_attn_kernel_choice", "rs_tmap_cache_stats")
LIN_EPILOGUE = {"bias": 0, "gelu": 1, "residual": 2}
KERNEL_CLASSES = ("layernorm", "gemm", "attn", "score", "select", "gather")


class RsError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


class AttnDesc(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int), ("B", ctypes.c_int), ("N", ctypes.c_int), ("H", ctypes.c_int),
                ("head_dim", ctypes.c_int), ("scale", ctypes.c_float),
                ("q_batch_stride", ctypes.c_longlong), ("q_row_stride", ctypes.c_longlong),
                ("q_head_stride", ctypes.c_longlong),
                ("k_batch_stride", ctypes.c_longlong), ("k_row_stride", ctypes.c_longlong),
                ("k_head_stride", ctypes.c_longlong),
                ("v_batch_stride", ctypes.c_longlong), ("v_row_stride", ctypes.c_longlong),
                ("v_head_stride", ctypes.c_longlong)]


class BlockDesc(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int), ("out_dtype", ctypes.c_int), ("B", ctypes.c_int),
                ("N", ctypes.c_int), ("D", ctypes.c_int), ("H", ctypes.c_int), ("D_mlp", ctypes.c_int),
                ("r", ctypes.c_int), ("has_cls", ctypes.c_int), ("ln_eps", ctypes.c_float),
                ("scale", ctypes.c_float), ("score_mode", ctypes.c_int), ("dist", ctypes.c_int)]


class VitDesc(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int), ("B", ctypes.c_int), ("N", ctypes.c_int), ("D", ctypes.c_int),
                ("H", ctypes.c_int), ("D_mlp", ctypes.c_int), ("L", ctypes.c_int), ("has_cls", ctypes.c_int),
                ("ln_eps", ctypes.c_float), ("scale", ctypes.c_float), ("score_mode", ctypes.c_int),
                ("dist", ctypes.c_int)]


class VitTaps(ctypes.Structure):
    """Host arrays of L device pointers (or NULL): every block's x_out, scores, keep_idx."""
    _fields_ = [("x_out", ctypes.POINTER(ctypes.c_void_p)), ("scores", ctypes.POINTER(ctypes.c_void_p)),
                ("keep_idx", ctypes.POINTER(ctypes.c_void_p))]


class BlockWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("w_qkv", "w_o", "w_fc1", "w_fc2", "b_qkv", "b_o", "b_fc1", "b_fc2",
                 "ln1_g", "ln1_b", "ln2_g", "ln2_b", "w_qkv_ln", "c_qkv_ln", "b_qkv_ln")]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load librs.so (built in-tree by paper_2508_00367_b200.build).  Fails loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_00367_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.rs_create.argtypes = [ctypes.POINTER(vp), ci]
    lib.rs_create.restype = ci
    lib.rs_destroy.argtypes = [vp]
    lib.rs_destroy.restype = None
    lib.rs_last_error.argtypes = [vp]
    lib.rs_last_error.restype = ctypes.c_char_p
    lib.rs_async_status.argtypes = [vp, vp]
    lib.rs_async_status.restype = ci
    lib.rs_uses_tensor_cores.argtypes = [vp, ci]
    lib.rs_uses_tensor_cores.restype = ci
    lib.rs_launch_count.argtypes = [vp]
    lib.rs_launch_count.restype = ctypes.c_longlong
    lib.rs_timing_enable.argtypes = [vp, ci]
    lib.rs_timing_enable.restype = ci
    lib.rs_timing_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong)]
    lib.rs_timing_read.restype = ci
    lib.rs_attn_fwd.argtypes = [vp, ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp]
    lib.rs_attn_fwd.restype = ci
    lib.rs_shift_score.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp, vp]
    lib.rs_shift_score.restype = ci
    lib.rs_topk_compact.argtypes = [vp, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp]
    lib.rs_topk_compact.restype = ci
    lib.rs_linewise_compact.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp]
    lib.rs_linewise_compact.restype = ci
    lib.rs_block_workspace_bytes.argtypes = [ctypes.POINTER(BlockDesc)]
    lib.rs_block_workspace_bytes.restype = ctypes.c_size_t
    lib.rs_block_fwd.argtypes = [vp, ctypes.POINTER(BlockDesc), ctypes.POINTER(BlockWeights), vp, vp, vp, vp,
                                 vp, vp, ctypes.c_size_t, vp]
    lib.rs_block_fwd.restype = ci
    lib.rs_linear_fwd.argtypes = [vp, ci, ci, ctypes.c_longlong, ci, ci, vp, vp, vp, vp, vp, vp]
    lib.rs_linear_fwd.restype = ci
    lib.rs_static_scratch_bytes.argtypes = []
    lib.rs_static_scratch_bytes.restype = ctypes.c_size_t
    lib.rs_block_fwd_static.argtypes = [ctypes.POINTER(BlockDesc), ctypes.POINTER(BlockWeights), vp, vp, vp, vp, vp,
                                        vp, ctypes.c_char_p, ctypes.c_size_t]
    lib.rs_block_fwd_static.restype = ci
    lib.rs_static_async_status.argtypes = [vp, ctypes.c_char_p, ctypes.c_size_t]
    lib.rs_static_async_status.restype = ci
    lib.rs_linear_uses_tensor_cores.argtypes = [vp, ci, ctypes.c_longlong, ci, ci]
    lib.rs_linear_uses_tensor_cores.restype = ci
    lib.rs_block_uses_tensor_cores.argtypes = [vp, ctypes.POINTER(BlockDesc)]
    lib.rs_block_uses_tensor_cores.restype = ci
    lib.rs_tmap_cache_stats.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ctypes.c_longlong)]
    lib.rs_tmap_cache_stats.restype = ci
    lib.rs_attn_fwd_ragged.argtypes = [vp, ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp]
    lib.rs_attn_fwd_ragged.restype = ci
    lib.rs_topk_compact_ragged.argtypes = [vp, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.rs_topk_compact_ragged.restype = ci
    lib.rs_block_fwd_ragged.argtypes = [vp, ctypes.POINTER(BlockDesc), ctypes.POINTER(BlockWeights), vp, vp, vp, vp, vp,
                                        vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.rs_block_fwd_ragged.restype = ci
    lib.rs_vit_workspace_bytes.argtypes = [ctypes.POINTER(VitDesc), ctypes.POINTER(ci)]
    lib.rs_vit_workspace_bytes.restype = ctypes.c_size_t
    lib.rs_vit_fwd.argtypes = [vp, ctypes.POINTER(VitDesc), ctypes.POINTER(BlockWeights), ctypes.POINTER(ci), vp, vp, vp,
                               vp, vp, ctypes.c_size_t, vp]
    lib.rs_vit_fwd.restype = ci
    lib.rs_vit_fwd_taps.argtypes = [vp, ctypes.POINTER(VitDesc), ctypes.POINTER(BlockWeights), ctypes.POINTER(ci), vp,
                                    ctypes.POINTER(VitTaps), vp, ctypes.c_size_t, vp]
    lib.rs_vit_fwd_taps.restype = ci
    lib.rs_vit_fwd_ragged.argtypes = [vp, ctypes.POINTER(VitDesc), ctypes.POINTER(BlockWeights), ctypes.POINTER(ci), vp, vp, vp,
                                      vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.rs_vit_fwd_ragged.restype = ci
    lib.rs_prepare_ln1_fold.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.rs_prepare_ln1_fold.restype = ci
    lib.rs_attn_kernel_choice.argtypes = [ci, ci, ci, ci]
    lib.rs_attn_kernel_choice.restype = ci
    _lib = lib
    return lib


def attn_kernel_choice(sm_count: int, B: int, H: int, N: int) -> int:
    """rs_attn_kernel_choice: 2 or 3, the attention kernel rs_attn_fwd picks for the shape (host arithmetic only)."""
    return int(load_library().rs_attn_kernel_choice(sm_count, B, H, N))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return RS_BF16
    if t.dtype == torch.float32:
        return RS_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _torch_dt(code: int):
    return torch.bfloat16 if code == RS_BF16 else torch.float32


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


class Context:
    """One rs_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the library has no CPU path")
        self.device = torch.device("cuda", device)
        h = ctypes.c_void_p()
        st = self.lib.rs_create(ctypes.byref(h), device)
        if st != RS_OK:
            raise RsError(st, "rs_create failed")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self.lib.rs_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != RS_OK:
            raise RsError(st, self.lib.rs_last_error(self.handle).decode())

    def raw(self, fn: str, *args) -> int:
        """Call an entry point with pre-marshalled arguments; returns the status code."""
        return getattr(self.lib, fn)(self.handle, *args)

    def last_error(self) -> str:
        return self.lib.rs_last_error(self.handle).decode()

    def async_status(self):
        self._check(self.lib.rs_async_status(self.handle, _stream(self.device)))

    def uses_tensor_cores(self, dtype=torch.bfloat16) -> bool:
        return bool(self.lib.rs_uses_tensor_cores(self.handle, RS_BF16 if dtype == torch.bfloat16 else RS_F32))

    def block_uses_tensor_cores(self, desc: "BlockDesc") -> bool:
        return bool(self.lib.rs_block_uses_tensor_cores(self.handle, ctypes.byref(desc)))

    def linear_uses_tensor_cores(self, dtype, M: int, N: int, K: int) -> bool:
        return bool(self.lib.rs_linear_uses_tensor_cores(self.handle, RS_BF16 if dtype == torch.bfloat16 else RS_F32, M, N, K))

    def tmap_cache_stats(self):
        """(hits, misses) of the context's tensor-map cache."""
        h, m = ctypes.c_longlong(), ctypes.c_longlong()
        self._check(self.lib.rs_tmap_cache_stats(self.handle, ctypes.byref(h), ctypes.byref(m)))
        return int(h.value), int(m.value)

    def launch_count(self) -> int:
        return int(self.lib.rs_launch_count(self.handle))

    def timing_enable(self, on: bool):
        self._check(self.lib.rs_timing_enable(self.handle, int(on)))

    def timing_read(self) -> Dict[str, Dict[str, float]]:
        """Per-kernel-class device time (ms) and launch count since the last read."""
        ms = (ctypes.c_double * len(KERNEL_CLASSES))()
        n = (ctypes.c_longlong * len(KERNEL_CLASSES))()
        self._check(self.lib.rs_timing_read(self.handle, _stream(self.device), ms, n))
        return {k: dict(ms=float(ms[i]), launches=int(n[i])) for i, k in enumerate(KERNEL_CLASSES)}

    # ---- rs_attn_fwd ----
    def attn_fwd(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float = 0.0,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q, k, v: [B, N, H, 64] views (innermost contiguous).  Returns [B, N, H*64]."""
        B, N, H, dh = q.shape
        for t in (q, k, v):
            assert t.is_cuda and t.stride(3) == 1 and t.shape == q.shape and t.dtype == q.dtype
        if out is None:
            out = torch.empty(B, N, H * dh, dtype=q.dtype, device=q.device)
        d = AttnDesc(_dt(q), B, N, H, dh, float(scale),
                     q.stride(0), q.stride(1), q.stride(2), k.stride(0), k.stride(1), k.stride(2),
                     v.stride(0), v.stride(1), v.stride(2))
        self._check(self.lib.rs_attn_fwd(self.handle, ctypes.byref(d), _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                         _stream(q.device)))
        return out

    # ---- per-sample token counts (padded layout) ----
    def attn_fwd_ragged(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens: torch.Tensor,
                        scale: float = 0.0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """rs_attn_fwd_ragged: sample b attends over its first seq_lens[b] tokens; rows behind them are unspecified."""
        B, N, H, dh = q.shape
        assert seq_lens.dtype == torch.int32 and seq_lens.is_cuda and seq_lens.numel() == B
        if out is None:
            out = torch.zeros(B, N, H * dh, dtype=q.dtype, device=q.device)
        d = AttnDesc(_dt(q), B, N, H, dh, float(scale),
                     q.stride(0), q.stride(1), q.stride(2), k.stride(0), k.stride(1), k.stride(2),
                     v.stride(0), v.stride(1), v.stride(2))
        self._check(self.lib.rs_attn_fwd_ragged(self.handle, ctypes.byref(d), _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                                _ptr(seq_lens), _stream(q.device)))
        return out

    def topk_compact_ragged(self, scores: torch.Tensor, x: Optional[torch.Tensor], seq_lens: torch.Tensor,
                            drops: torch.Tensor, K_pad: int, has_cls: bool = True):
        """rs_topk_compact_ragged -> (x_out [B, K_pad, D] or None, keep_idx [B, K_pad], lens_out [B])."""
        B, N = scores.shape
        dev = scores.device
        keep_idx = torch.empty(B, K_pad, dtype=torch.int32, device=dev)
        lens_out = torch.empty(B, dtype=torch.int32, device=dev)
        D, dt, x_out = 8, RS_F32, None
        if x is not None:
            D, dt = x.shape[2], _dt(x)
            x_out = torch.empty(B, K_pad, D, dtype=x.dtype, device=dev)
        self._check(self.lib.rs_topk_compact_ragged(self.handle, dt, B, N, D, K_pad, int(has_cls), _ptr(scores), _ptr(x),
                                                    _ptr(x_out), _ptr(keep_idx), _ptr(seq_lens), _ptr(drops),
                                                    _ptr(lens_out), _stream(dev)))
        return x_out, keep_idx, lens_out

    def block_fwd_ragged(self, x: torch.Tensor, weights: "DeviceBlockWeights", H: int, seq_lens: torch.Tensor,
                         drops: torch.Tensor, K_pad: int, has_cls: bool = True, out_dtype=None,
                         want_full: bool = False) -> Dict[str, torch.Tensor]:
        """rs_block_fwd_ragged on a padded batch.  Returns dict(x_out [B, K_pad, D], scores [B, N], keep_idx
        [B, K_pad], lens_out [B][, x_full])."""
        assert x.is_cuda and x.is_contiguous()
        B, N, D = x.shape
        desc = self.block_desc(B, N, D, H, weights.D_mlp, N - K_pad, x.dtype, out_dtype, has_cls)
        odt = _torch_dt(desc.out_dtype)
        ws = torch.empty(max(self.block_workspace_bytes(desc), 256), dtype=torch.uint8, device=x.device)
        res = dict(x_out=torch.empty(B, K_pad, D, dtype=odt, device=x.device),
                   scores=torch.empty(B, N, dtype=torch.float32, device=x.device),
                   keep_idx=torch.empty(B, K_pad, dtype=torch.int32, device=x.device),
                   lens_out=torch.empty(B, dtype=torch.int32, device=x.device))
        x_full = torch.empty(B, N, D, dtype=odt, device=x.device) if want_full else None
        self._check(self.lib.rs_block_fwd_ragged(self.handle, ctypes.byref(desc), ctypes.byref(weights.struct), _ptr(x),
                                                 _ptr(res["x_out"]), _ptr(res["scores"]), _ptr(res["keep_idx"]), _ptr(x_full),
                                                 _ptr(seq_lens), _ptr(drops), _ptr(res["lens_out"]), _ptr(ws), ws.numel(),
                                                 _stream(x.device)))
        if want_full:
            res["x_full"] = x_full
        return res

    def vit_fwd_ragged(self, x: torch.Tensor, weights: Sequence["DeviceBlockWeights"], H: int, pad_drops: Sequence[int],
                       seq_lens: torch.Tensor, sample_drops: torch.Tensor, has_cls: bool = True) -> Dict[str, torch.Tensor]:
        """rs_vit_fwd_ragged: the layer loop on a padded batch with per-sample token counts.  sample_drops is
        [L, B] int32 on the device.  Returns dict(x_out [B, N_L, D], keep_idx [B, N_L], lens_out [B])."""
        assert x.is_cuda and x.is_contiguous() and len(weights) == len(pad_drops)
        B, N, D = x.shape
        L = len(weights)
        assert sample_drops.dtype == torch.int32 and sample_drops.is_contiguous() and tuple(sample_drops.shape) == (L, B)
        assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
        desc = VitDesc(_dt(x), B, N, D, H, weights[0].D_mlp, L, int(has_cls), 0.0, 0.0, SCORE_MODE["mlp"], DIST["l2"])
        cdrops = (ctypes.c_int * L)(*[int(r) for r in pad_drops])
        warr = (BlockWeights * L)(*[w.struct for w in weights])
        need = int(self.lib.rs_vit_workspace_bytes(ctypes.byref(desc), cdrops))
        if need == 0:
            raise RsError(1, "rs_vit_fwd_ragged: bad descriptor or schedule")
        ws = torch.empty(need, dtype=torch.uint8, device=x.device)
        n_out = N - sum(int(r) for r in pad_drops)
        res = dict(x_out=torch.empty(B, n_out, D, dtype=x.dtype, device=x.device),
                   keep_idx=torch.empty(B, n_out, dtype=torch.int32, device=x.device),
                   lens_out=torch.empty(B, dtype=torch.int32, device=x.device))
        self._check(self.lib.rs_vit_fwd_ragged(self.handle, ctypes.byref(desc), warr, cdrops, _ptr(x), _ptr(res["x_out"]),
                                               _ptr(res["keep_idx"]), _ptr(seq_lens), _ptr(sample_drops), _ptr(res["lens_out"]),
                                               _ptr(ws), ws.numel(), _stream(x.device)))
        return res

    # ---- rs_linear_fwd ----
    def linear_fwd(self, a: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                   epilogue: str = "bias", residual: Optional[torch.Tensor] = None) -> torch.Tensor:
        """out = epilogue(a @ w.T + bias); a [M, K], w [N, K]; fp32 output for the residual epilogue."""
        M, K = a.shape
        N = w.shape[0]
        assert a.is_contiguous() and w.is_contiguous() and w.shape[1] == K and w.dtype == a.dtype
        out = torch.empty(M, N, dtype=torch.float32 if epilogue == "residual" else a.dtype, device=a.device)
        self._check(self.lib.rs_linear_fwd(self.handle, _dt(a), LIN_EPILOGUE[epilogue], M, N, K, _ptr(a), _ptr(w),
                                           _ptr(bias), _ptr(residual), _ptr(out), _stream(a.device)))
        return out

    # ---- rs_shift_score ----
    def shift_score(self, after: torch.Tensor, before: torch.Tensor, dist: str = "l2",
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B, N, D = after.shape
        assert after.is_contiguous() and before.is_contiguous() and before.shape == after.shape
        if out is None:
            out = torch.empty(B, N, dtype=torch.float32, device=after.device)
        self._check(self.lib.rs_shift_score(self.handle, _dt(after), DIST[dist], B, N, D, _ptr(after),
                                            _ptr(before), _ptr(out), _stream(after.device)))
        return out

    # ---- rs_topk_compact ----
    def topk_compact(self, scores: torch.Tensor, x: Optional[torch.Tensor], r: int, has_cls: bool = True,
                     x_out: Optional[torch.Tensor] = None, keep_idx: Optional[torch.Tensor] = None):
        B, N = scores.shape
        K = N - r
        assert scores.dtype == torch.float32 and scores.is_contiguous()
        if keep_idx is None:
            keep_idx = torch.empty(B, max(K, 0), dtype=torch.int32, device=scores.device)
        D = 8
        dt = RS_F32
        if x is not None:
            assert x.is_contiguous() and x.shape[:2] == (B, N)
            D = x.shape[2]
            dt = _dt(x)
            if x_out is None:
                x_out = torch.empty(B, max(K, 0), D, dtype=x.dtype, device=x.device)
        self._check(self.lib.rs_topk_compact(self.handle, dt, B, N, D, r, int(has_cls), _ptr(scores), _ptr(x),
                                             _ptr(x_out), _ptr(keep_idx), _stream(scores.device)))
        return x_out, keep_idx

    # ---- rs_linewise_compact ----
    def linewise_compact(self, scores: torch.Tensor, x: Optional[torch.Tensor], drop_rows: int, drop_cols: int,
                         x_out: Optional[torch.Tensor] = None, keep_rows: Optional[torch.Tensor] = None,
                         keep_cols: Optional[torch.Tensor] = None):
        """scores [B, H, W] fp32, x [B, H, W, D] or None -> (x_out or None, keep_rows, keep_cols)."""
        B, H, W = scores.shape
        assert scores.dtype == torch.float32 and scores.is_contiguous()
        if keep_rows is None:
            keep_rows = torch.empty(B, max(H - drop_rows, 0), dtype=torch.int32, device=scores.device)
        if keep_cols is None:
            keep_cols = torch.empty(B, max(W - drop_cols, 0), dtype=torch.int32, device=scores.device)
        D, dt = 8, RS_F32
        if x is not None:
            assert x.is_contiguous() and tuple(x.shape[:3]) == (B, H, W)
            D, dt = x.shape[3], _dt(x)
            if x_out is None:
                x_out = torch.empty(B, max(H - drop_rows, 0), max(W - drop_cols, 0), D, dtype=x.dtype, device=x.device)
        self._check(self.lib.rs_linewise_compact(self.handle, dt, B, H, W, D, drop_rows, drop_cols, _ptr(scores), _ptr(x),
                                                 _ptr(x_out), _ptr(keep_rows), _ptr(keep_cols), _stream(scores.device)))
        return x_out, keep_rows, keep_cols

    # ---- rs_vit_fwd ----
    def vit_fwd(self, x: torch.Tensor, weights: Sequence["DeviceBlockWeights"], H: int, drops: Sequence[int],
                has_cls: bool = True, score_mode: str = "mlp", dist: str = "l2",
                workspace: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
        """The whole layer loop in one library call.  Returns dict(x_out, scores, keep_idx) of the last block."""
        assert x.is_cuda and x.is_contiguous() and len(weights) == len(drops)
        B, N, D = x.shape
        L = len(weights)
        desc = VitDesc(_dt(x), B, N, D, H, weights[0].D_mlp, L, int(has_cls), 0.0, 0.0, SCORE_MODE[score_mode], DIST[dist])
        cdrops = (ctypes.c_int * L)(*[int(r) for r in drops])
        warr = (BlockWeights * L)(*[w.struct for w in weights])
        need = int(self.lib.rs_vit_workspace_bytes(ctypes.byref(desc), cdrops))
        if need == 0:
            raise RsError(1, "rs_vit_fwd: bad descriptor or schedule")
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        n_last = N - sum(int(r) for r in drops[:-1])
        n_out = n_last - int(drops[-1])
        x_out = torch.empty(B, n_out, D, dtype=x.dtype, device=x.device)
        scores = torch.empty(B, n_last, dtype=torch.float32, device=x.device)
        keep = torch.empty(B, n_out, dtype=torch.int32, device=x.device)
        self._check(self.lib.rs_vit_fwd(self.handle, ctypes.byref(desc), warr, cdrops, _ptr(x), _ptr(x_out), _ptr(scores),
                                        _ptr(keep), _ptr(workspace), workspace.numel(), _stream(x.device)))
        return dict(x_out=x_out, scores=scores, keep_idx=keep)

    def vit_fwd_taps(self, x: torch.Tensor, weights: Sequence["DeviceBlockWeights"], H: int, drops: Sequence[int],
                     tap_blocks: Sequence[int], has_cls: bool = True, score_mode: str = "mlp",
                     dist: str = "l2") -> Dict[int, Dict[str, torch.Tensor]]:
        """rs_vit_fwd_taps with outputs requested for the blocks in `tap_blocks` only (the last block is
        always included); the other blocks' tokens live in the call's workspace.  Returns
        {block: dict(x_out, scores, keep_idx)}."""
        assert x.is_cuda and x.is_contiguous() and len(weights) == len(drops)
        B, N, D = x.shape
        L = len(weights)
        desc = VitDesc(_dt(x), B, N, D, H, weights[0].D_mlp, L, int(has_cls), 0.0, 0.0, SCORE_MODE[score_mode], DIST[dist])
        cdrops = (ctypes.c_int * L)(*[int(r) for r in drops])
        warr = (BlockWeights * L)(*[w.struct for w in weights])
        need = int(self.lib.rs_vit_workspace_bytes(ctypes.byref(desc), cdrops))
        if need == 0:
            raise RsError(1, "rs_vit_fwd: bad descriptor or schedule")
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        want = set(int(b) for b in tap_blocks) | {L - 1}
        outs, n = {}, N
        arrs = {k: (ctypes.c_void_p * L)() for k in ("x_out", "scores", "keep_idx")}
        for l, r in enumerate(drops):
            k = n - int(r)
            if l in want:
                outs[l] = dict(x_out=torch.empty(B, k, D, dtype=x.dtype, device=x.device),
                               scores=torch.empty(B, n, dtype=torch.float32, device=x.device),
                               keep_idx=torch.empty(B, k, dtype=torch.int32, device=x.device))
                for key in arrs:
                    arrs[key][l] = outs[l][key].data_ptr()
            n = k
        taps = VitTaps(arrs["x_out"], arrs["scores"], arrs["keep_idx"])
        self._check(self.lib.rs_vit_fwd_taps(self.handle, ctypes.byref(desc), warr, cdrops, _ptr(x), ctypes.byref(taps),
                                             _ptr(workspace), workspace.numel(), _stream(x.device)))
        return outs

    # ---- rs_block_fwd ----
    def block_desc(self, B, N, D, H, D_mlp, r, dtype, out_dtype=None, has_cls=True, ln_eps=0.0, scale=0.0,
                   score_mode="mlp", dist="l2") -> BlockDesc:
        code = RS_BF16 if dtype == torch.bfloat16 else RS_F32
        ocode = code if out_dtype is None else (RS_BF16 if out_dtype == torch.bfloat16 else RS_F32)
        return BlockDesc(code, ocode, B, N, D, H, D_mlp, r, int(has_cls), float(ln_eps), float(scale),
                         SCORE_MODE[score_mode], DIST[dist])

    def block_workspace_bytes(self, desc: BlockDesc) -> int:
        return int(self.lib.rs_block_workspace_bytes(ctypes.byref(desc)))

    def block_fwd(self, x: torch.Tensor, weights: "DeviceBlockWeights", H: int, r: int, has_cls: bool = True,
                  out_dtype=None, score_mode: str = "mlp", ln_eps: float = 0.0, scale: float = 0.0,
                  want_full: bool = False, workspace: Optional[torch.Tensor] = None,
                  x_out: Optional[torch.Tensor] = None, scores: Optional[torch.Tensor] = None,
                  keep_idx: Optional[torch.Tensor] = None, dist: str = "l2") -> Dict[str, torch.Tensor]:
        """One block + pruning.  Returns dict(x_out, scores, keep_idx[, x_full])."""
        assert x.is_cuda and x.is_contiguous()
        B, N, D = x.shape
        desc = self.block_desc(B, N, D, H, weights.D_mlp, r, x.dtype, out_dtype, has_cls, ln_eps, scale, score_mode, dist)
        odt = _torch_dt(desc.out_dtype)
        K = N - r
        need = self.block_workspace_bytes(desc)
        if workspace is None:
            workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
        if x_out is None:
            x_out = torch.empty(B, max(K, 0), D, dtype=odt, device=x.device)
        if scores is None:
            scores = torch.empty(B, N, dtype=torch.float32, device=x.device)
        if keep_idx is None:
            keep_idx = torch.empty(B, max(K, 0), dtype=torch.int32, device=x.device)
        x_full = torch.empty(B, N, D, dtype=odt, device=x.device) if want_full else None
        self._check(self.lib.rs_block_fwd(self.handle, ctypes.byref(desc), ctypes.byref(weights.struct), _ptr(x),
                                          _ptr(x_out), _ptr(scores), _ptr(keep_idx), _ptr(x_full),
                                          _ptr(workspace), workspace.numel(), _stream(x.device)))
        res = dict(x_out=x_out, scores=scores, keep_idx=keep_idx)
        if want_full:
            res["x_full"] = x_full
        return res


def block_fwd_static(x: torch.Tensor, weights: "DeviceBlockWeights", H: int, r: int, has_cls: bool = True,
                     out_dtype=None, score_mode: str = "mlp", want_full: bool = False):
    """rs_block_fwd_static: the block without a context or a workspace, for callers that
    may not allocate device memory at the point of the call.  Scratch is the library's
    built-in array (rs_static_scratch_bytes()); larger blocks raise RsError(RS_ERR_WORKSPACE).
    Calls sharing a device must be serialised on one stream.  The output tensors made
    here are ordinary torch allocations -- a caller that cannot allocate passes its own
    buffers through the C ABI directly."""
    lib = load_library()
    B, N, D = x.shape
    code = _dt(x)
    ocode = code if out_dtype is None else (RS_BF16 if out_dtype == torch.bfloat16 else RS_F32)
    desc = BlockDesc(code, ocode, B, N, D, H, weights.D_mlp, r, int(has_cls), 0.0, 0.0, SCORE_MODE[score_mode], 0)
    K = N - r
    odt = _torch_dt(ocode)
    x_out = torch.empty(B, max(K, 0), D, dtype=odt, device=x.device)
    scores = torch.empty(B, N, dtype=torch.float32, device=x.device)
    keep_idx = torch.empty(B, max(K, 0), dtype=torch.int32, device=x.device)
    x_full = torch.empty(B, N, D, dtype=odt, device=x.device) if want_full else None
    err = ctypes.create_string_buffer(512)
    with torch.cuda.device(x.device):
        st = lib.rs_block_fwd_static(ctypes.byref(desc), ctypes.byref(weights.struct), _ptr(x), _ptr(x_out),
                                     _ptr(scores), _ptr(keep_idx), _ptr(x_full), _stream(x.device), err, 512)
    if st != RS_OK:
        raise RsError(st, err.value.decode())
    res = dict(x_out=x_out, scores=scores, keep_idx=keep_idx)
    if want_full:
        res["x_full"] = x_full
    return res


def static_async_status(device) -> None:
    """rs_static_async_status: synchronise the current stream of `device` and raise if a kernel of an
    earlier block_fwd_static call reported a device-side anomaly."""
    lib = load_library()
    err = ctypes.create_string_buffer(512)
    with torch.cuda.device(device):
        st = lib.rs_static_async_status(_stream(device), err, 512)
    if st != RS_OK:
        raise RsError(st, err.value.decode())


class DeviceBlockWeights:
    """Block parameters resident on the device: matrices in the storage dtype,
    biases and LayerNorm parameters in fp32."""

    MATS = ("w_qkv", "w_o", "w_fc1", "w_fc2")
    VECS = ("b_qkv", "b_o", "b_fc1", "b_fc2", "ln1_g", "ln1_b", "ln2_g", "ln2_b")

    def __init__(self, w: Dict[str, torch.Tensor], dtype: torch.dtype, device):
        self.t = {}
        for n in self.MATS:
            self.t[n] = w[n].to(device=device, dtype=dtype).contiguous()
        for n in self.VECS:
            self.t[n] = None if w.get(n) is None else w[n].to(device=device, dtype=torch.float32).contiguous()
        self.D_mlp = self.t["w_fc1"].shape[0]
        self.struct = BlockWeights(*[None if self.t[n] is None else self.t[n].data_ptr()
                                     for n in self.MATS + self.VECS])

    def fold_ln1(self, ctx: "Context"):
        """rs_prepare_ln1_fold: LN1 folded into the QKV weights (bf16 only), for the layer loop."""
        w = self.t["w_qkv"]
        assert w.dtype == torch.bfloat16
        D = w.shape[1]
        self.t["w_qkv_ln"] = torch.empty_like(w)
        self.t["c_qkv_ln"] = torch.empty(3 * D, dtype=torch.float32, device=w.device)
        self.t["b_qkv_ln"] = torch.empty(3 * D, dtype=torch.float32, device=w.device)
        ctx._check(ctx.lib.rs_prepare_ln1_fold(ctx.handle, RS_BF16, D, _ptr(w), _ptr(self.t["b_qkv"]), _ptr(self.t["ln1_g"]),
                                               _ptr(self.t["ln1_b"]), _ptr(self.t["w_qkv_ln"]), _ptr(self.t["c_qkv_ln"]),
                                               _ptr(self.t["b_qkv_ln"]), _stream(w.device)))
        for n in ("w_qkv_ln", "c_qkv_ln", "b_qkv_ln"):
            setattr(self.struct, n, self.t[n].data_ptr())


class PrunedViT:
    """Layer loop of the pruned forward pass: block l+1 consumes block l's
    compacted output; `drops[l]` tokens are removed after block l."""

    def __init__(self, ctx: Context, blocks: Sequence[Dict[str, torch.Tensor]], H: int, drops: Sequence[int],
                 dtype: torch.dtype, has_cls: bool = True, score_mode: str = "mlp", dist: str = "l2",
                 tap_blocks: Optional[Sequence[int]] = None, fold_ln1: bool = False):
        """tap_blocks: the blocks whose compacted tokens x_out the caller wants (the last block always);
        None = every block.  A pruning block that is not tapped writes no dense copy of its kept
        tokens: the next block reads them in place through the index list.  Scores and kept indices
        are returned for every tapped block and for every block that drops tokens."""
        assert len(blocks) == len(drops)
        self.ctx, self.H, self.drops, self.dtype = ctx, H, list(drops), dtype
        L = len(self.drops)
        self.tapped = set(range(L)) if tap_blocks is None else (set(int(b) for b in tap_blocks) | {L - 1})
        self.has_cls, self.score_mode, self.dist = has_cls, score_mode, dist
        self.weights: List[DeviceBlockWeights] = [DeviceBlockWeights(w, dtype, ctx.device) for w in blocks]
        if fold_ln1 and dtype == torch.bfloat16 and self.weights[0].t["w_qkv"].shape[1] % 128 == 0:
            # LN1 of every block but the first is applied inside its QKV product
            for l in range(1, L):
                self.weights[l].fold_ln1(ctx)
        self._plan = None

    def plan(self, B: int, N: int, D: int):
        """Allocate the workspace and the per-block outputs once for a shape."""
        key = (B, N, D)
        if self._plan and self._plan["key"] == key:
            return self._plan
        dev = self.ctx.device
        L = len(self.drops)
        outs, n = [], N
        for l, r in enumerate(self.drops):
            k = n - r
            o = {}
            if l in self.tapped or r > 0:
                o = dict(scores=torch.empty(B, n, dtype=torch.float32, device=dev),
                         keep_idx=torch.empty(B, k, dtype=torch.int32, device=dev))
            if l in self.tapped:
                o["x_out"] = torch.empty(B, k, D, dtype=self.dtype, device=dev)
            outs.append(o)
            n = k
        code = RS_BF16 if self.dtype == torch.bfloat16 else RS_F32
        desc = VitDesc(code, B, N, D, self.H, self.weights[0].D_mlp, L, int(self.has_cls), 0.0, 0.0,
                       SCORE_MODE[self.score_mode], DIST[self.dist])
        cdrops = (ctypes.c_int * L)(*[int(r) for r in self.drops])
        warr = (BlockWeights * L)(*[w.struct for w in self.weights])
        need = int(self.ctx.lib.rs_vit_workspace_bytes(ctypes.byref(desc), cdrops))
        if need == 0:
            raise RsError(1, "rs_vit_fwd: bad descriptor or schedule")
        arrs = {k: (ctypes.c_void_p * L)(*[(o[k].data_ptr() if k in o else None) for o in outs])
                for k in ("x_out", "scores", "keep_idx")}
        taps = VitTaps(arrs["x_out"], arrs["scores"], arrs["keep_idx"])
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
        self._plan = dict(key=key, desc=desc, drops=cdrops, warr=warr, arrs=arrs, taps=taps, outs=outs, ws=ws)
        return self._plan

    def forward(self, x: torch.Tensor, graph: bool = False):
        """x: [B, N, D] on the device.  Returns the list of per-block outputs (buffers owned by
        the plan and overwritten by the next call).

        graph=True replays the whole layer loop as one CUDA graph, captured on first use for
        this input buffer (the graph reads x at its address: pass the same tensor again, or a
        few fixed ones).  The first call for a shape must come outside any capture: it runs the
        loop once eagerly so that every kernel's one-time set-up has happened."""
        B, N, D = x.shape
        p = self.plan(B, N, D)
        if not graph:
            self._run(x, p)
            return p["outs"]
        graphs = p.setdefault("graphs", {})
        key = (x.data_ptr(), torch.cuda.current_stream(x.device).cuda_stream)
        g = graphs.get(key)
        if g is None:
            if not p.get("warm"):
                self._run(x, p)
                torch.cuda.synchronize(x.device)
                p["warm"] = True
            n0 = self.ctx.launch_count()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._run(x, p)
            p["launches_per_forward"] = self.ctx.launch_count() - n0
            graphs[key] = (g, x)          # keep x alive: the graph holds its address
            g = graphs[key]
        g[0].replay()
        return p["outs"]

    def launches_per_forward(self, B: int, N: int, D: int) -> int:
        """Kernels one forward pass launches (known once a graph was captured for the shape)."""
        return int(self.plan(B, N, D).get("launches_per_forward", 0))

    def _run(self, x: torch.Tensor, p):
        """One library call: the layer loop with every block's outputs written to the plan's buffers."""
        rc = self.ctx.lib.rs_vit_fwd_taps(self.ctx.handle, ctypes.byref(p["desc"]), p["warr"], p["drops"], _ptr(x),
                                          ctypes.byref(p["taps"]), _ptr(p["ws"]), p["ws"].numel(), _stream(x.device))
        if rc != RS_OK:
            raise RsError(rc, self.ctx.last_error())
