"""ctypes loader for the CPU oracle (``rib_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
module.  It compiles the C file with gcc on first use and wraps its functions with numpy
``float64`` arrays.  Nothing here is shared with, or imported by, the CUDA path.

The arithmetic lives in ``rib_oracle.c`` (Eq. 5 and Eq. 6 of the paper, SoftMax(S)V, and the
chain rule of that definition); this file only marshals arguments.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
# RIB_ORACLE_SRC points the loader at another C file; the mutation test uses it to check that
# the pins fail on a deliberately broken copy of the oracle.
_SRC = Path(os.environ.get("RIB_ORACLE_SRC", _HERE / "rib_oracle.c"))
_LIB = (_HERE / "_build" / "librib_oracle.so" if "RIB_ORACLE_SRC" not in os.environ
        else _SRC.with_suffix(".so"))
_lock = threading.Lock()
_lib = None

_c_dp = ctypes.POINTER(ctypes.c_double)
_c_lp = ctypes.POINTER(ctypes.c_long)


def build(force: bool = False) -> Path:
    """Compile rib_oracle.c into a shared library next to it (gcc -O2 -fopenmp, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall",
             str(_SRC), "-o", str(tmp), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(str(build()))
            lib.rib_oracle_fwd.restype = ctypes.c_int
            lib.rib_oracle_fwd.argtypes = [_c_dp] * 5 + [ctypes.c_int] * 8 + [
                ctypes.c_long, _c_lp, ctypes.c_long, _c_dp, _c_dp]
            lib.rib_oracle_bwd.restype = ctypes.c_int
            lib.rib_oracle_bwd.argtypes = [_c_dp] * 6 + [ctypes.c_int] * 8 + [
                ctypes.c_long, _c_lp, ctypes.c_long] + [_c_dp] * 5
            lib.rib_oracle_pair_matrices.restype = ctypes.c_int
            lib.rib_oracle_pair_matrices.argtypes = [_c_dp] * 6 + [ctypes.c_int] * 8 + [
                ctypes.c_long, ctypes.c_long, _c_dp, _c_dp]
            lib.rib_oracle_token_pixel.restype = None
            lib.rib_oracle_token_pixel.argtypes = [ctypes.c_int] * 7 + [
                ctypes.POINTER(ctypes.c_int)] * 2
            lib.rib_oracle_num_pairs.restype = ctypes.c_int
            lib.rib_oracle_num_pairs.argtypes = [ctypes.c_int] * 5
            lib.rib_oracle_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_c_dp)


def _pairs_arg(pairs):
    if pairs is None:
        return None, None, 0
    arr = np.ascontiguousarray(np.asarray(pairs, dtype=np.int64))
    return arr, arr.ctypes.data_as(_c_lp), arr.size


def _p_shape(pq, n, r, heads):
    pq = np.asarray(pq)
    if pq.shape == (n, r):
        return 0
    if pq.shape == (heads, n, r):
        return n * r
    raise ValueError(f"pq/pk must be [n={n}, r={r}] or [heads, n, r], got {pq.shape}")


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().rib_oracle_threads())


def num_pairs(B, H, W, heads, window) -> int:
    return int(_load().rib_oracle_num_pairs(B, H, W, heads, window))


def token_pixel(H, W, window, shift, wy, wx, i):
    """Image pixel (Y, X) of token i of window (wy, wx) under cyclic shift."""
    Y, X = ctypes.c_int(), ctypes.c_int()
    _load().rib_oracle_token_pixel(H, W, window, shift, wy, wx, i, ctypes.byref(Y), ctypes.byref(X))
    return Y.value, X.value


def fwd(q, k, v, pq, pk, window, shift=0, pairs=None):
    """out [B,H,W,heads,d] and lse [B,heads,H,W] in float64.

    q, k, v: [B,H,W,heads,d]; pq, pk: [n,r] or [heads,n,r].  With ``pairs`` (flat pair ids) only
    those pairs are computed and the remaining entries are NaN.
    """
    q = _f64(q)
    B, H, W, heads, d = q.shape
    k, v = _f64(k, q.shape), _f64(v, q.shape)
    n = window * window
    r = np.asarray(pq).shape[-1]
    stride = _p_shape(pq, n, r, heads)
    pq, pk = _f64(pq), _f64(pk, np.asarray(pq).shape)
    out = np.full(q.shape, np.nan)
    lse = np.full((B, heads, H, W), np.nan)
    keep, pptr, np_ = _pairs_arg(pairs)
    rc = _load().rib_oracle_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), B, H, W, heads, d,
                                r, window, shift, stride, pptr, np_, _ptr(out), _ptr(lse))
    if rc:
        raise ValueError(f"rib_oracle_fwd rejected the shape (code {rc})")
    return out, lse


def bwd(q, k, v, pq, pk, dout, window, shift=0, pairs=None):
    """dq, dk, dv [B,H,W,heads,d] and dpq, dpk (shape of pq) in float64.

    With ``pairs`` only those pairs are processed: untouched dq/dk/dv entries are NaN and
    dpq/dpk are the sums over the listed pairs only.
    """
    q = _f64(q)
    B, H, W, heads, d = q.shape
    k, v, dout = _f64(k, q.shape), _f64(v, q.shape), _f64(dout, q.shape)
    n = window * window
    r = np.asarray(pq).shape[-1]
    stride = _p_shape(pq, n, r, heads)
    pq, pk = _f64(pq), _f64(pk, np.asarray(pq).shape)
    dq, dk, dv = (np.full(q.shape, np.nan) for _ in range(3))
    dpq, dpk = np.zeros(pq.shape), np.zeros(pq.shape)
    keep, pptr, np_ = _pairs_arg(pairs)
    rc = _load().rib_oracle_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), _ptr(dout), B, H, W,
                                heads, d, r, window, shift, stride, pptr, np_, _ptr(dq), _ptr(dk),
                                _ptr(dv), _ptr(dpq), _ptr(dpk))
    if rc:
        raise ValueError(f"rib_oracle_bwd rejected the shape (code {rc})")
    return dq, dk, dv, dpq, dpk


def pair_matrices(q, k, v, pq, pk, dout, window, shift, pid):
    """Probability matrix P and logit gradient dS (both [n,n]) of one pair; dS is None without dout."""
    q = _f64(q)
    B, H, W, heads, d = q.shape
    k, v = _f64(k, q.shape), _f64(v, q.shape)
    dout = None if dout is None else _f64(dout, q.shape)
    n = window * window
    r = np.asarray(pq).shape[-1]
    stride = _p_shape(pq, n, r, heads)
    pq, pk = _f64(pq), _f64(pk, np.asarray(pq).shape)
    P = np.empty((n, n))
    dS = np.empty((n, n)) if dout is not None else None
    rc = _load().rib_oracle_pair_matrices(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), _ptr(dout),
                                          B, H, W, heads, d, r, window, shift, stride, pid,
                                          _ptr(P), _ptr(dS))
    if rc:
        raise ValueError(f"rib_oracle_pair_matrices rejected the shape (code {rc})")
    return P, dS
