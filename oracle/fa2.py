"""CPU oracle for the FlashAttention-2 recurrence (per-query running maximum, normaliser and output over key tiles).

TEST INFRASTRUCTURE ONLY.  Written in C (``cyc_oracle_fa2.c``, fp64) from the recurrence of Section "Simulated Cholesky
and Flash Attention"; called through ctypes with numpy arrays.  It shares nothing with the CUDA library and must not be
imported by the product package.

``Q`` is ``[N][d]``, ``K`` and ``V`` are ``[M][d]`` (float32, or uint16 holding bf16 bit patterns, widened here exactly);
results are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcyc_oracle_fa2.so")
_SOURCE = os.path.join(_HERE, "cyc_oracle_fa2.c")
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-pthread"]
ERRORS = {1: "bad argument", 2: "out of memory"}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_SOURCE) > os.path.getmtime(_LIB_PATH):
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SOURCE, "-lm"], cwd=_HERE)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _widen(x):
    x = np.asarray(x)
    if x.dtype == np.uint16:  # bf16 bit patterns: the top half of a float32
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return np.ascontiguousarray(x, dtype=np.float32)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def attention(Q, K, V, tile: int, *, threads: int = 1, with_state: bool = False):
    """Run the recurrence over key tiles of ``tile`` rows.

    Returns ``O`` or, with ``with_state``, ``(O, m, l, A)``: the final running maximum and normaliser of every query and
    ``A[i][c] = sum_j softmax_ij |V_jc|``."""
    Q, K, V = np.ascontiguousarray(_widen(Q)), np.ascontiguousarray(_widen(K)), np.ascontiguousarray(_widen(V))
    if Q.ndim != 2 or K.ndim != 2 or V.shape != K.shape or K.shape[1] != Q.shape[1]:
        raise ValueError("Q must be [N][d], K and V [M][d]")
    N, d = Q.shape
    M = K.shape[0]
    O = np.empty((N, d), dtype=np.float64)
    m = np.empty(N, dtype=np.float64) if with_state else None
    l = np.empty(N, dtype=np.float64) if with_state else None
    A = np.empty((N, d), dtype=np.float64) if with_state else None
    i64 = ctypes.c_int64
    rc = lib().cyc_oracle_fa2(i64(N), i64(M), i64(d), i64(int(tile)), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(m), _ptr(l),
                              _ptr(A), int(threads))
    if rc:
        raise RuntimeError("fa2 oracle: " + ERRORS.get(rc, "error %d" % rc))
    return (O, m, l, A) if with_state else O
