"""CPU oracle for the prefix-sum recurrence ``P_i = P_{i-1} + A_i`` (Figure "Representative recurrences").

TEST INFRASTRUCTURE ONLY.  Written in C (``cyc_oracle_scan.c``): the recurrence walked one element at a time in
increasing ``i`` from ``P_{-1} = 0``; called through ctypes with numpy arrays.  It shares nothing with the CUDA library
and must not be imported by the product package.

``A`` is ``[n]`` or ``[rows][n]`` (rows are independent sequences); float32 or int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcyc_oracle_scan.so")
_SOURCE = os.path.join(_HERE, "cyc_oracle_scan.c")
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC"]


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


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _shape(A):
    if A.ndim == 1:
        return 1, A.shape[0]
    if A.ndim == 2:
        return A.shape
    raise ValueError("A must be [n] or [rows][n]")


def prefix_sum(A, *, arithmetic: str = "f64", with_scale: bool = False):
    """Walk the recurrence over every row of ``A``.

    ``arithmetic``: ``"f64"`` (float32 input, running value in fp64; the reference of the tolerance checks), ``"f32"``
    (running value in fp32) or ``"i32"`` (wrapping 32-bit integers).  With ``with_scale`` (f64 only) also returns
    ``S_i = sum_{k<=i} |A_k|``."""
    i64 = ctypes.c_int64
    if arithmetic == "i32":
        A = np.ascontiguousarray(A, dtype=np.int32)
        rows, n = _shape(A)
        P = np.empty_like(A)
        rc = lib().cyc_oracle_prefix_sum_i32(i64(rows), i64(n), i64(n), _ptr(A), _ptr(P))
        S = None
    elif arithmetic == "f32":
        A = np.ascontiguousarray(A, dtype=np.float32)
        rows, n = _shape(A)
        P = np.empty_like(A)
        rc = lib().cyc_oracle_prefix_sum_f32(i64(rows), i64(n), i64(n), _ptr(A), _ptr(P))
        S = None
    elif arithmetic == "f64":
        A = np.ascontiguousarray(A, dtype=np.float32)
        rows, n = _shape(A)
        P = np.empty(A.shape, dtype=np.float64)
        S = np.empty(A.shape, dtype=np.float64) if with_scale else None
        rc = lib().cyc_oracle_prefix_sum_f64(i64(rows), i64(n), i64(n), _ptr(A), _ptr(P), _ptr(S))
    else:
        raise ValueError("arithmetic must be f64, f32 or i32")
    if rc:
        raise RuntimeError("scan oracle: bad argument")
    return (P, S) if with_scale else P
