"""ctypes front end of the fp64 CPU oracle (oracle/rs_oracle.c).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's cpu_baseline / reference arm may import this module.  It imports
nothing from the CUDA package and the CUDA package imports nothing from here.

All tensors are NumPy float64 arrays, C-contiguous.  Rounding to the storage
type of the GPU interface (bf16 or fp32) is applied only to tensors that cross
that interface: block inputs and outputs, attention q/k/v/out, score inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rs_oracle.c")
_LIB = os.path.join(_HERE, "liborc.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c99",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_num_threads.restype = ctypes.c_int
        _lib.orc_topk.restype = ctypes.c_int
        _lib.orc_block_fwd.restype = ctypes.c_int
        _lib.orc_linewise.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_dp)


def _dopt(a):
    if a is None:
        return None, None
    return _d(a)


# ---- rounding to the interface storage type (Eq.-free: IEEE round-to-nearest-even) ----

def round_bf16(a) -> np.ndarray:
    """fp64 -> nearest bf16 (ties to even), returned as fp64.  Goes through fp32
    first, as the GPU does when it narrows an fp32 accumulator."""
    f = np.ascontiguousarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    nan = np.isnan(f)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = u.astype(np.uint32).view(np.float32).astype(np.float64)
    out[nan] = np.nan
    return out


def round_f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64).astype(np.float32).astype(np.float64)


def round_to(a, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_bf16(a)
    if dtype == "f32":
        return round_f32(a)
    if dtype == "f64":
        return np.ascontiguousarray(a, dtype=np.float64)
    raise ValueError(dtype)


# ---- the parts ----

def layernorm(x, gamma, beta, eps=1e-6):
    x, xp = _d(x)
    D = x.shape[-1]
    T = x.size // D
    g, gp = _d(gamma)
    b, bp = _d(beta)
    out = np.empty_like(x)
    _load().orc_layernorm(xp, gp, bp, ctypes.c_double(eps), ctypes.c_long(T), ctypes.c_int(D),
                          out.ctypes.data_as(_dp))
    return out


def linear(x, W, bias=None):
    x, xp = _d(x)
    W, Wp = _d(W)
    out_f, in_f = W.shape
    assert x.shape[-1] == in_f
    T = x.size // in_f
    b, bp = _dopt(bias)
    y = np.empty(x.shape[:-1] + (out_f,), dtype=np.float64)
    _load().orc_linear(xp, Wp, bp, ctypes.c_long(T), ctypes.c_int(in_f), ctypes.c_int(out_f),
                       y.ctypes.data_as(_dp))
    return y


def gelu(x):
    y = np.array(x, dtype=np.float64, order="C", copy=True)
    _load().orc_gelu(y.ctypes.data_as(_dp), ctypes.c_long(y.size))
    return y


def attn(q, k, v, scale=None):
    """Eq. sa per (sample, head).  q, k, v: [B, N, H, dh] (any strides)."""
    q, qp = _d(q)
    k, kp = _d(k)
    v, vp = _d(v)
    B, N, H, dh = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(dh)
    out = np.empty_like(q)
    _load().orc_attn(qp, kp, vp, ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(H),
                     ctypes.c_int(dh), ctypes.c_double(scale), out.ctypes.data_as(_dp))
    return out


DIST = {"l2": 0, "l1": 1, "cos": 2}
SCORE_MODE = {"mlp": 0, "mlp_delta": 1, "attn": 2, "block": 3}


def shift_score(after, before, dist="l2"):
    a, ap = _d(after)
    b, bp = _d(before)
    assert a.shape == b.shape
    D = a.shape[-1]
    T = a.size // D
    s = np.empty(a.shape[:-1], dtype=np.float64)
    _load().orc_shift_score(ap, bp, ctypes.c_long(T), ctypes.c_int(D), ctypes.c_int(DIST[dist]),
                            s.ctypes.data_as(_dp))
    return s


def topk(scores, r, has_cls=True):
    s, sp = _d(scores)
    B, N = s.shape
    K = N - r
    keep = np.empty((B, max(K, 0)), dtype=np.int32)
    rc = _load().orc_topk(sp, ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(r),
                          ctypes.c_int(int(has_cls)), keep.ctypes.data_as(_ip))
    if rc != 0:
        raise ValueError("r must satisfy 0 <= r <= N-1")
    return keep


def gather(x, keep_idx):
    x, xp = _d(x)
    B, N, D = x.shape
    keep = np.ascontiguousarray(keep_idx, dtype=np.int32)
    K = keep.shape[1]
    out = np.empty((B, K, D), dtype=np.float64)
    _load().orc_gather(xp, keep.ctypes.data_as(_ip), ctypes.c_int(B), ctypes.c_int(N),
                       ctypes.c_int(K), ctypes.c_int(D), out.ctypes.data_as(_dp))
    return out


def linewise(scores, drop_rows, drop_cols):
    """Sec. 4 (CNN, line-wise variant): scores [B, H, W] -> (keep_rows [B, H - drop_rows],
    keep_cols [B, W - drop_cols]), the lines whose average shift is not among the lowest."""
    s, sp = _d(scores)
    B, H, W = s.shape
    kr = np.empty((B, max(H - drop_rows, 0)), dtype=np.int32)
    kc = np.empty((B, max(W - drop_cols, 0)), dtype=np.int32)
    rc = _load().orc_linewise(sp, ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(W), ctypes.c_int(drop_rows),
                              ctypes.c_int(drop_cols), kr.ctypes.data_as(_ip), kc.ctypes.data_as(_ip))
    if rc != 0:
        raise ValueError("drop counts must leave at least one row and one column")
    return kr, kc


def grid_gather(x, keep_rows, keep_cols):
    """x [B, H, W, D] -> [B, Hk, Wk, D]: the rows and columns that are kept."""
    x, xp = _d(x)
    B, H, W, D = x.shape
    kr = np.ascontiguousarray(keep_rows, dtype=np.int32)
    kc = np.ascontiguousarray(keep_cols, dtype=np.int32)
    Hk, Wk = kr.shape[1], kc.shape[1]
    out = np.empty((B, Hk, Wk, D), dtype=np.float64)
    _load().orc_grid_gather(xp, kr.ctypes.data_as(_ip), kc.ctypes.data_as(_ip), ctypes.c_int(B), ctypes.c_int(H),
                            ctypes.c_int(W), ctypes.c_int(Hk), ctypes.c_int(Wk), ctypes.c_int(D),
                            out.ctypes.data_as(_dp))
    return out


WEIGHT_NAMES = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


def block_fwd(x, w: dict, H: int, r: int, has_cls=True, eps=1e-6, scale=None,
              score_mode="mlp", dist="l2", forced_keep=None):
    """One block + pruning (Eq. att, Eq. MLP, Sec. 3.2).  `w` maps WEIGHT_NAMES to
    arrays (Linear weights are [out, in]).  Returns a dict with x_prime, m,
    x_hat, scores, keep_idx, x_out (all fp64 / int32, unrounded).  With
    `forced_keep` the gather uses those indices instead of the oracle's own."""
    x, xp = _d(x)
    B, N, D = x.shape
    Dm = np.asarray(w["w_fc1"]).shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(D // H)
    K = N - r
    arrs = {}
    ptrs = []
    for name in WEIGHT_NAMES:
        a, p = _dopt(w.get(name))
        arrs[name] = a
        ptrs.append(p)
    x_prime = np.empty_like(x)
    m = np.empty_like(x)
    x_hat = np.empty_like(x)
    scores = np.empty((B, N), dtype=np.float64)
    keep = np.empty((B, K), dtype=np.int32)
    x_out = np.empty((B, K, D), dtype=np.float64)
    rc = _load().orc_block_fwd(
        xp, ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(D), ctypes.c_int(H), ctypes.c_int(Dm),
        *ptrs,
        ctypes.c_double(eps), ctypes.c_double(scale), ctypes.c_int(SCORE_MODE[score_mode]),
        ctypes.c_int(DIST[dist]), ctypes.c_int(r), ctypes.c_int(int(has_cls)),
        x_prime.ctypes.data_as(_dp), m.ctypes.data_as(_dp), x_hat.ctypes.data_as(_dp),
        scores.ctypes.data_as(_dp), keep.ctypes.data_as(_ip), x_out.ctypes.data_as(_dp))
    if rc != 0:
        raise ValueError("r must satisfy 0 <= r <= N-1")
    if forced_keep is not None:
        keep = np.ascontiguousarray(forced_keep, dtype=np.int32)
        x_out = gather(x_hat, keep)
    return dict(x_prime=x_prime, m=m, x_hat=x_hat, scores=scores, keep_idx=keep, x_out=x_out)


def model_fwd(x, blocks, H, drops, has_cls=True, eps=1e-6, io_dtype="bf16",
              score_mode="mlp", dist="l2", forced_keeps=None):
    """Layer loop: block l+1 consumes block l's x_out rounded to the interface
    storage type.  `drops[l]` = tokens removed after block l (0-based list, one
    entry per block).  Returns the per-block result dicts (x_out already
    rounded under key 'x_out_rounded')."""
    cur = round_to(x, io_dtype)
    outs = []
    for l, w in enumerate(blocks):
        fk = None if forced_keeps is None else forced_keeps[l]
        res = block_fwd(cur, w, H, drops[l], has_cls=has_cls, eps=eps, score_mode=score_mode,
                        dist=dist, forced_keep=fk)
        res["x_out_rounded"] = round_to(res["x_out"], io_dtype)
        outs.append(res)
        cur = res["x_out_rounded"]
    return outs
