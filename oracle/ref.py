"""ctypes front end of the C oracle (test infrastructure only).

The arithmetic lives in ``topk_oracle.c``; this module compiles it with gcc
(no CUDA involved), loads it and converts numpy arrays to pointers.  It shares
nothing with the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "topk_oracle.c")
_LIB = os.path.join(_HERE, "libtopk_oracle.so")
_lib = None

# Contraction must stay off so that p*v and alpha*s are rounded before the
# add/subtract (two roundings per term), and no fast-math reassociation.
_CFLAGS = ["-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC", "-pthread"]
_LDLIBS = ["-lm"]


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC, *_LDLIBS], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, i32p, f32p, u8p = ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        lib.ref_topk.argtypes = [f32p, i64, i64, i32p, f32p]
        lib.ref_topk.restype = ctypes.c_int
        lib.ref_topk_rows.argtypes = [f32p, i64, i64, i64, i32p, f32p, ctypes.c_int]
        lib.ref_topk_rows.restype = ctypes.c_int
        lib.ref_aggregate.argtypes = [i32p, f32p, i64, i64, f32p, i64, f32p, u8p]
        lib.ref_aggregate.restype = ctypes.c_int
        lib.ref_step.argtypes = [f32p, f32p, i64, i64, i64, i64, f32p, ctypes.c_float, ctypes.c_int,
                                 i32p, f32p, f32p, u8p, i32p, f32p, ctypes.c_void_p, ctypes.c_int]
        lib.ref_step.restype = ctypes.c_int
        lib.ref_rho.argtypes = [f32p, f32p, f32p, i64, i64, i64, i64, f32p, ctypes.c_float, ctypes.c_int, ctypes.c_int]
        lib.ref_rho.restype = ctypes.c_double
        lib.ref_lost_energy.argtypes = [f32p, i64, i32p, i64]
        lib.ref_lost_energy.restype = ctypes.c_double
        lib.ref_step_ef.argtypes = [f32p, f32p, f32p, f32p, i64, i64, i64, i64, f32p, ctypes.c_float, ctypes.c_int,
                                    i32p, f32p, i32p, f32p, ctypes.c_void_p, ctypes.c_int]
        lib.ref_step_ef.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def ref_topk(x, K: int):
    """Top_K of one vector: (idx int32[K] ascending, val float32[K])."""
    x = _f32(x).reshape(-1)
    idx = np.empty(K, dtype=np.int32)
    val = np.empty(K, dtype=np.float32)
    rc = _load().ref_topk(_ptr(x), x.size, K, _ptr(idx), _ptr(val))
    if rc != 0:
        raise ValueError("ref_topk rejected its arguments (d=%d, K=%d)" % (x.size, K))
    return idx, val


def ref_topk_rows(x, K: int, nthreads: Optional[int] = None):
    """Top_K of every row of x[rows][d]: (idx int32[rows][K], val float32[rows][K])."""
    x = _f32(x)
    assert x.ndim == 2
    rows, d = x.shape
    idx = np.empty((rows, K), dtype=np.int32)
    val = np.empty((rows, K), dtype=np.float32)
    nt = default_threads() if nthreads is None else nthreads
    rc = _load().ref_topk_rows(_ptr(x), rows, d, K, _ptr(idx), _ptr(val), nt)
    if rc != 0:
        raise ValueError("ref_topk_rows rejected its arguments")
    return idx, val


def ref_aggregate(up_idx, up_val, p, d: int):
    """Ordered weighted sum of N sparse messages: (A float32[d], touched uint8[d])."""
    up_idx = np.ascontiguousarray(up_idx, dtype=np.int32)
    up_val = _f32(up_val)
    p = _f32(p)
    N, K_up = up_idx.shape
    A = np.empty(d, dtype=np.float32)
    touched = np.empty(d, dtype=np.uint8)
    rc = _load().ref_aggregate(_ptr(up_idx), _ptr(up_val), N, K_up, _ptr(p), d, _ptr(A), _ptr(touched))
    if rc != 0:
        raise ValueError("ref_aggregate rejected its arguments")
    return A, touched


@dataclass
class StepResult:
    w: np.ndarray          # updated parameters
    up_idx: np.ndarray     # [N][K_up]
    up_val: np.ndarray     # [N][K_up]
    A: np.ndarray          # dense aggregate [d]
    touched: np.ndarray    # uint8[d]
    msg_idx: np.ndarray    # downlink message indices, ascending
    msg_val: np.ndarray    # downlink message values


def ref_step(w, G, K_up: int, K_down: int, p, alpha: float, mode: int,
             nthreads: Optional[int] = None, want_dense: bool = True) -> StepResult:
    """One memory-free iteration; returns the new w and every intermediate."""
    w = _f32(w).copy()
    G = _f32(G)
    p = _f32(p)
    N, d = G.shape
    assert w.shape == (d,) and p.shape == (N,)
    up_idx = np.empty((N, K_up), dtype=np.int32)
    up_val = np.empty((N, K_up), dtype=np.float32)
    A = np.empty(d, dtype=np.float32) if want_dense else None
    touched = np.empty(d, dtype=np.uint8) if want_dense else None
    cap = min(d, K_down if mode == 1 else N * K_up)
    msg_idx = np.empty(cap, dtype=np.int32)
    msg_val = np.empty(cap, dtype=np.float32)
    count = ctypes.c_int64(0)
    nt = default_threads() if nthreads is None else nthreads
    rc = _load().ref_step(_ptr(w), _ptr(G), N, d, K_up, K_down, _ptr(p), ctypes.c_float(alpha), mode,
                          _ptr(up_idx), _ptr(up_val), _ptr(A), _ptr(touched),
                          _ptr(msg_idx), _ptr(msg_val), ctypes.byref(count), nt)
    if rc != 0:
        raise ValueError("ref_step rejected its arguments")
    n = count.value
    return StepResult(w, up_idx, up_val, A, touched, msg_idx[:n].copy(), msg_val[:n].copy())


@dataclass
class EfResult:
    w: np.ndarray          # updated parameters
    eps: np.ndarray        # updated worker memories [N][d]
    delta: Optional[np.ndarray]  # updated server memory [d] (bidirectional)
    up_idx: np.ndarray
    up_val: np.ndarray
    msg_idx: np.ndarray
    msg_val: np.ndarray


def ref_step_ef(w, eps, delta, G, K_up: int, K_down: int, p, alpha: float, mode: int,
                nthreads: Optional[int] = None) -> EfResult:
    """One iteration of Algorithm 1 (mode 0) / Algorithm 2 (mode 1) with the error memories.
    Inputs are not modified; the new w, eps, delta are returned."""
    w = _f32(w).copy()
    eps = _f32(eps).copy()
    G = _f32(G)
    p = _f32(p)
    N, d = G.shape
    assert w.shape == (d,) and eps.shape == (N, d) and p.shape == (N,)
    if mode == 1:
        delta = _f32(delta).copy()
        assert delta.shape == (d,)
    else:
        delta = None
    up_idx = np.empty((N, K_up), dtype=np.int32)
    up_val = np.empty((N, K_up), dtype=np.float32)
    cap = min(d, K_down if mode == 1 else N * K_up)
    msg_idx = np.empty(cap, dtype=np.int32)
    msg_val = np.empty(cap, dtype=np.float32)
    count = ctypes.c_int64(0)
    nt = default_threads() if nthreads is None else nthreads
    rc = _load().ref_step_ef(_ptr(w), _ptr(eps), _ptr(delta), _ptr(G), N, d, K_up, K_down, _ptr(p),
                             ctypes.c_float(alpha), mode, _ptr(up_idx), _ptr(up_val),
                             _ptr(msg_idx), _ptr(msg_val), ctypes.byref(count), nt)
    if rc != 0:
        raise ValueError("ref_step_ef rejected its arguments")
    n = count.value
    return EfResult(w, eps, delta, up_idx, up_val, msg_idx[:n].copy(), msg_val[:n].copy())


def ref_lost_energy(x, idx) -> float:
    """||Top_K(x) - x||^2 / ||x||^2 for the message with indices idx (the appendix's 1 - gamma)."""
    x = _f32(x).reshape(-1)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    return float(_load().ref_lost_energy(_ptr(x), x.size, _ptr(idx), idx.size))


def ref_rho(G, eps, delta, K_up: int, K_down: int, p, alpha: float, mode: int,
            nthreads: Optional[int] = None) -> float:
    """The gap constant of one iteration: rho_hat (mode 0) or rho (mode 1).  eps / delta are the
    memories before the iteration; None = memory-free (then the step size cancels)."""
    G = _f32(G)
    p = _f32(p)
    N, d = G.shape
    eps = None if eps is None else _f32(eps)
    delta = None if delta is None else _f32(delta)
    nt = default_threads() if nthreads is None else nthreads
    r = _load().ref_rho(_ptr(G), _ptr(eps), _ptr(delta), N, d, K_up, K_down, _ptr(p), ctypes.c_float(alpha), mode, nt)
    if r < 0:
        raise ValueError("ref_rho rejected its arguments")
    return float(r)
