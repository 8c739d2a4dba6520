"""ctypes front end of the C oracle (TEST INFRASTRUCTURE ONLY).

The arithmetic lives in ``attention_oracle.c`` (Eq. 1 of the paper, written as
three plain fp64 passes per query row).  This module only compiles that file
with gcc, loads it and marshals numpy arrays; it holds no arithmetic itself.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attention_oracle.c")
_LIB = os.path.join(_HERE, "libattention_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 -march=native -fopenmp); return the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared",
                   "-std=c99", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        path = build()
        lib = ctypes.CDLL(path)
        vp, i32, i64p, dp, f64 = (ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_double)
        lib.oracle_attention.restype = ctypes.c_int
        lib.oracle_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32,
                                         i32, f64, i64p, ctypes.c_int64, dp, dp, i32]
        lib.oracle_attention_prow.restype = ctypes.c_int
        lib.oracle_attention_prow.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32,
                                              i32, f64, i32, i32, i32, dp, dp, dp]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle uses by default (OpenMP's maximum)."""
    return int(_load().oracle_num_threads())


def _prepare(Q, K, V):
    Q = np.ascontiguousarray(Q)
    K = np.ascontiguousarray(K)
    V = np.ascontiguousarray(V)
    if Q.ndim != 4 or K.ndim != 4 or V.ndim != 4:
        raise ValueError("Q, K, V must be [B,H,S,d] arrays")
    if Q.dtype == np.float64 and K.dtype == np.float64 and V.dtype == np.float64:
        kind = 0
    elif Q.dtype == np.uint16 and K.dtype == np.uint16 and V.dtype == np.uint16:
        kind = 1  # bf16 bit patterns
    else:
        raise TypeError("inputs must be all float64 or all uint16 (bf16 bit patterns)")
    B, Hq, Sq, dqk = Q.shape
    Bk, Hkv, Sk, dk2 = K.shape
    Bv, Hv, Sv, dv = V.shape
    if not (B == Bk == Bv and Hkv == Hv and Sk == Sv and dqk == dk2):
        raise ValueError("inconsistent Q/K/V shapes")
    return Q, K, V, kind, (B, Hq, Hkv, Sq, Sk, dqk, dv)


def attention(Q, K, V, *, causal: bool, scale: float, rows=None, threads: int = 0):
    """O, lse of softmax(scale * Q K^T [+ causal mask]) V in fp64.

    Q [B,Hq,Sq,dqk], K [B,Hkv,Sk,dqk], V [B,Hkv,Sk,dv]: float64, or uint16 holding
    bf16 bit patterns.  ``rows`` = optional int array [n,3] of (b, hq, i); then
    O is [n,dv] and lse [n].  Otherwise O is [B,Hq,Sq,dv] and lse [B,Hq,Sq].
    """
    Q, K, V, kind, (B, Hq, Hkv, Sq, Sk, dqk, dv) = _prepare(Q, K, V)
    lib = _load()
    if rows is not None:
        rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64).reshape(-1, 3))
        n = rows.shape[0]
        O = np.empty((n, dv), dtype=np.float64)
        lse = np.empty((n,), dtype=np.float64)
        rows_p = rows.ctypes.data
    else:
        n = 0
        O = np.empty((B, Hq, Sq, dv), dtype=np.float64)
        lse = np.empty((B, Hq, Sq), dtype=np.float64)
        rows_p = None
    rc = lib.oracle_attention(Q.ctypes.data, K.ctypes.data, V.ctypes.data, kind,
                              B, Hq, Hkv, Sq, Sk, dqk, dv, int(bool(causal)), float(scale),
                              rows_p, n, O.ctypes.data, lse.ctypes.data, int(threads))
    if rc != 0:
        raise ValueError("oracle_attention failed with code %d" % rc)
    return O, lse


def attention_prow(Q, K, V, *, causal: bool, scale: float, b: int, hq: int, i: int):
    """Probabilities P[i, :] (zeros where masked), the O row and lse of one query row."""
    Q, K, V, kind, (B, Hq, Hkv, Sq, Sk, dqk, dv) = _prepare(Q, K, V)
    lib = _load()
    P = np.empty((Sk,), dtype=np.float64)
    O = np.empty((dv,), dtype=np.float64)
    lse = ctypes.c_double(0.0)
    rc = lib.oracle_attention_prow(Q.ctypes.data, K.ctypes.data, V.ctypes.data, kind,
                                   B, Hq, Hkv, Sq, Sk, dqk, dv, int(bool(causal)), float(scale),
                                   int(b), int(hq), int(i), P.ctypes.data, O.ctypes.data,
                                   ctypes.byref(lse))
    if rc != 0:
        raise ValueError("oracle_attention_prow failed with code %d" % rc)
    return P, O, float(lse.value)
