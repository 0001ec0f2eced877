"""ctypes front end of the fp64 C oracle (oracle/bigla_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU-baseline / reference legs, never by the product path.

Every function takes numpy arrays that already hold the exact input values
(fp64 copies of the stored bf16 / fp32 numbers) in the dense row-major
[B, H, L, d] layout, and returns fp64 results.  The arithmetic lives in the C
file; this module only builds it with gcc and marshals pointers.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bigla_oracle.c")
_LIB = os.path.join(_HERE, "libbigla_oracle.so")
_lock = threading.Lock()
_handle = None


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle with gcc (plain -O2, no fast-math) and return the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm", "-lpthread"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _lib():
    global _handle
    if _handle is None:
        path = build_oracle()
        lib = ctypes.CDLL(path)
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_bigla_fwd.argtypes = [dp] * 8 + [ctypes.c_long] * 5 + [ctypes.c_int]
        lib.oracle_bigla_fwd.restype = ctypes.c_int
        lib.oracle_gate_prep.argtypes = [dp, dp, ctypes.c_long, ctypes.c_double]
        lib.oracle_gate_prep.restype = ctypes.c_int
        _handle = lib
    return _handle


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def bigla_fwd_directions(q, k, v, log_alpha_fwd, log_alpha_bwd, nthreads: int = 1):
    """Eq. 6 by the plain recurrence.  Returns (o, o_fwd, o_bwd, threads_used)."""
    q = _f64(q)
    if q.ndim != 4:
        raise ValueError("q must be [B, H, L, dk]")
    B, H, L, dk = q.shape
    k = _f64(k, (B, H, L, dk))
    la_f = _f64(log_alpha_fwd, (B, H, L, dk))
    la_b = _f64(log_alpha_bwd, (B, H, L, dk))
    v = _f64(v)
    if v.ndim != 4 or v.shape[:3] != (B, H, L):
        raise ValueError("v must be [B, H, L, dv]")
    dv = v.shape[3]
    out = np.zeros((B, H, L, dv), dtype=np.float64)
    out_f = np.zeros_like(out)
    out_b = np.zeros_like(out)
    used = _lib().oracle_bigla_fwd(
        _ptr(q), _ptr(k), _ptr(v), _ptr(la_f), _ptr(la_b),
        _ptr(out), _ptr(out_f), _ptr(out_b), B, H, L, dk, dv, int(nthreads),
    )
    if used < 0:
        raise RuntimeError("oracle_bigla_fwd rejected its arguments")
    return out, out_f, out_b, used


def bigla_fwd(q, k, v, log_alpha_fwd, log_alpha_bwd, nthreads: int = 1):
    """o = (o_fwd + o_bwd) / 2 of Eq. 6, fp64, shape [B, H, L, dv]."""
    return bigla_fwd_directions(q, k, v, log_alpha_fwd, log_alpha_bwd, nthreads)[0]


def gate_prep(g, tau: float = 16.0):
    """log alpha = logsigmoid(g) / tau (Eq. 5 line 1), fp64, same shape as g."""
    g = _f64(g)
    la = np.empty_like(g)
    if _lib().oracle_gate_prep(_ptr(g), _ptr(la), g.size, float(tau)) != 0:
        raise RuntimeError("oracle_gate_prep rejected its arguments")
    return la
