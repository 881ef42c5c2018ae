"""ctypes front end of oracle/moe_oracle.c (fp64 plain-loop CPU oracle).

TEST INFRASTRUCTURE ONLY.  Inputs may be torch tensors or numpy arrays of any float
dtype (bf16 included); they are widened exactly to float64 before the C code sees them.
Each wrapper names the passage of the paper its C function follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, strict IEEE: no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_oracle())
        i32p, f32p, f64p, ci = (ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float),
                                ctypes.POINTER(ctypes.c_double), ctypes.c_int)
        lib.moe_oracle_threads.restype = ci
        lib.moe_oracle_route.argtypes = [f32p, ci, ci, ci, ci, i32p, f64p]
        lib.moe_oracle_layout.argtypes = [i32p, ci, ci, ci, ci, i32p, i32p, i32p, i32p]
        lib.moe_oracle_fwd.argtypes = [f64p, i32p, f64p, f64p, f64p, ci, ci, ci, ci, ci, ci, f64p, f64p, f64p, f64p]
        lib.moe_oracle_bwd.argtypes = [f64p, f64p, i32p, f64p, f64p, f64p, ci, ci, ci, ci, ci, ci,
                                       f64p, f64p, f64p, f64p]
        lib.moe_oracle_swiglu_add.argtypes = [f64p, f64p, ci, ci, f64p, f64p]
        lib.moe_oracle_router_logits.argtypes = [f64p, f64p, ci, ci, ci, f64p]
        lib.moe_oracle_router_bwd.argtypes = [f32p, i32p, f64p, ci, ci, ci, ci, f64p]
        lib.moe_oracle_route_sigmoid.argtypes = [f32p, ci, ci, ci, ci, i32p, f64p]
        lib.moe_oracle_router_bwd_sigmoid.argtypes = [f32p, i32p, f64p, ci, ci, ci, ci, f64p]
        _lib = lib
    return _lib


def _np(a, dtype):
    """torch tensor / array -> contiguous numpy array of `dtype` (exact widening for floats)."""
    if hasattr(a, "detach"):
        import torch
        a = a.detach().to("cpu")
        if a.dtype == torch.bfloat16:
            a = a.to(torch.float32)
        a = a.numpy()
    return np.ascontiguousarray(a, dtype=dtype)


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def threads() -> int:
    return int(_load().moe_oracle_threads())


def route(logits, k: int, renorm: bool, gate: str = "softmax"):
    """Top-k routing scores (Section 2.2, router description).  gate = "softmax" (scores over all E experts) or
    "sigmoid" (per-expert scores).  -> ids int32 [T,k], w float64 [T,k]."""
    l = _np(logits, np.float32)
    T, E = l.shape
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    fn = {"softmax": _load().moe_oracle_route, "sigmoid": _load().moe_oracle_route_sigmoid}[gate]
    rc = fn(_p(l, ctypes.c_float), T, E, k, int(bool(renorm)),
                                  _p(ids, ctypes.c_int32), _p(w, ctypes.c_double))
    if rc:
        raise ValueError(f"moe_oracle_route failed ({rc})")
    return ids, w


def layout(ids, E: int, S: int = 0):
    """Dispatch layout (Section 2.2, Dispatch).  -> counts [E+S], offsets [E+S+1], row_of, src_of [T*(k+S)]."""
    ids = _np(ids, np.int32)
    T, k = ids.shape
    n = T * (k + S)
    counts = np.empty(E + S, np.int32)
    offsets = np.empty(E + S + 1, np.int32)
    row_of = np.empty(n, np.int32)
    src_of = np.empty(n, np.int32)
    rc = _load().moe_oracle_layout(_p(ids, ctypes.c_int32), T, E, k, S, _p(counts, ctypes.c_int32),
                                   _p(offsets, ctypes.c_int32), _p(row_of, ctypes.c_int32),
                                   _p(src_of, ctypes.c_int32))
    if rc:
        raise ValueError(f"moe_oracle_layout failed ({rc}): expert id out of range")
    return counts, offsets, row_of, src_of


def fwd(x, ids, w, W_gate_up, W_down, S: int = 0, save: bool = False):
    """Forward MoE-FFN (Section 2.2, five forward operators).  -> out float64 [T,d]
    (and, with save=True, per-slot H [T*(k+S),2F], A [.,F], Y [.,d])."""
    x = _np(x, np.float64)
    ids = _np(ids, np.int32)
    w = _np(w, np.float64)
    Wgu = _np(W_gate_up, np.float64)
    Wd = _np(W_down, np.float64)
    T, d = x.shape
    k = ids.shape[1]
    Ep, F2, d2 = Wgu.shape
    F = F2 // 2
    E = Ep - S
    assert d2 == d and Wd.shape == (Ep, d, F) and w.shape == ids.shape and ids.shape[0] == T
    out = np.empty((T, d), np.float64)
    n = T * (k + S)
    H = np.empty((n, 2 * F), np.float64) if save else None
    A = np.empty((n, F), np.float64) if save else None
    Y = np.empty((n, d), np.float64) if save else None
    dp = ctypes.c_double
    rc = _load().moe_oracle_fwd(_p(x, dp), _p(ids, ctypes.c_int32), _p(w, dp), _p(Wgu, dp), _p(Wd, dp),
                                T, d, E, k, S, F, _p(out, dp), _p(H, dp), _p(A, dp), _p(Y, dp))
    if rc:
        raise ValueError(f"moe_oracle_fwd failed ({rc})")
    return (out, H, A, Y) if save else out


def bwd(dout, x, ids, w, W_gate_up, W_down, S: int = 0):
    """Backward MoE-FFN (Section 2.2, seven backward operators).
    -> dx [T,d], dW_gate_up [E+S,2F,d], dW_down [E+S,d,F], d_w [T,k] (all float64)."""
    dout = _np(dout, np.float64)
    x = _np(x, np.float64)
    ids = _np(ids, np.int32)
    w = _np(w, np.float64)
    Wgu = _np(W_gate_up, np.float64)
    Wd = _np(W_down, np.float64)
    T, d = x.shape
    k = ids.shape[1]
    Ep, F2, _ = Wgu.shape
    F = F2 // 2
    E = Ep - S
    assert dout.shape == x.shape and Wd.shape == (Ep, d, F)
    dx = np.empty((T, d), np.float64)
    dWgu = np.empty_like(Wgu)
    dWd = np.empty_like(Wd)
    dw = np.empty((T, k), np.float64)
    dp = ctypes.c_double
    rc = _load().moe_oracle_bwd(_p(dout, dp), _p(x, dp), _p(ids, ctypes.c_int32), _p(w, dp), _p(Wgu, dp),
                                _p(Wd, dp), T, d, E, k, S, F, _p(dx, dp), _p(dWgu, dp), _p(dWd, dp), _p(dw, dp))
    if rc:
        raise ValueError(f"moe_oracle_bwd failed ({rc})")
    return dx, dWgu, dWd, dw


def swiglu_add(x, r):
    """SwiGLU + Add operator pair of the scheduling microbenchmarks (Section 6): x [M,2C] = gate | up halves,
    r [M,C].  -> s = silu(gate) * up [M,C], z = s + r [M,C] (float64)."""
    x = _np(x, np.float64)
    r = _np(r, np.float64)
    M, C2 = x.shape
    C = C2 // 2
    assert C2 == 2 * C and r.shape == (M, C)
    s = np.empty((M, C), np.float64)
    z = np.empty((M, C), np.float64)
    dp = ctypes.c_double
    rc = _load().moe_oracle_swiglu_add(_p(x, dp), _p(r, dp), M, C, _p(s, dp), _p(z, dp))
    if rc:
        raise ValueError(f"moe_oracle_swiglu_add failed ({rc})")
    return s, z


def router_logits(x, W_r):
    """Linear router scores (Section 2.2, router description): x [T,d], W_r [E,d] -> logits float64 [T,E]."""
    x = _np(x, np.float64)
    W = _np(W_r, np.float64)
    T, d = x.shape
    E = W.shape[0]
    assert W.shape == (E, d)
    out = np.empty((T, E), np.float64)
    rc = _load().moe_oracle_router_logits(_p(x, ctypes.c_double), _p(W, ctypes.c_double), T, d, E, _p(out, ctypes.c_double))
    if rc:
        raise ValueError(f"moe_oracle_router_logits failed ({rc})")
    return out


def router_fwd(x, W_r, k: int, renorm: bool, gate: str = "softmax"):
    """Router in the path: logits in fp64, rounded once to fp32 (the precision the CUDA path decides in), then
    `route`.  -> ids int32 [T,k], w float64 [T,k], logits float64 [T,E] (unrounded)."""
    logits = router_logits(x, W_r)
    ids, w = route(logits.astype(np.float32), k, renorm, gate)
    return ids, w, logits


def router_bwd(logits, ids, d_topk_w, renorm: bool, gate: str = "softmax"):
    """Gradient of the k routing scores w.r.t. the logits (softmax over all E, optional renormalisation over the
    selected experts; no gradient through the selection).  -> d_logits float64 [T,E]."""
    l = _np(logits, np.float32)
    ids = _np(ids, np.int32)
    g = _np(d_topk_w, np.float64)
    T, E = l.shape
    k = ids.shape[1]
    assert ids.shape == (T, k) and g.shape == (T, k)
    out = np.empty((T, E), np.float64)
    fn = {"softmax": _load().moe_oracle_router_bwd, "sigmoid": _load().moe_oracle_router_bwd_sigmoid}[gate]
    rc = fn(_p(l, ctypes.c_float), _p(ids, ctypes.c_int32), _p(g, ctypes.c_double), T, E, k,
                                       int(bool(renorm)), _p(out, ctypes.c_double))
    if rc:
        raise ValueError(f"moe_oracle_router_bwd failed ({rc})")
    return out
