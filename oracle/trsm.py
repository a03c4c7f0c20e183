"""CPU oracle for the block lower-triangular solve ``L X = B``.

TEST INFRASTRUCTURE ONLY.  Evaluates ``X_i = TRSM(L_ii, B_i - sum_{j<i} GEMM(L_ij, X_j))`` (Section "Multiple
Iteration Spaces", Figure "deps-tri-solve") in fp64, written in C (``cyc_oracle_trsm.c``) and called through ctypes with
numpy arrays.  It shares nothing with the CUDA library and must not be imported by the product package.

``L`` is ``[n][n]`` float32 (only the lower triangle is read), ``B`` is ``[n][m]`` float32, the result is ``[n][m]``
float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcyc_oracle_trsm.so")
_SOURCE = os.path.join(_HERE, "cyc_oracle_trsm.c")
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-pthread"]
MODES = {"literal": 0, "collapsed": 1}
ERRORS = {1: "bad argument", 2: "out of memory", 3: "copy invariant (i,j)_Xb == X_j violated"}


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


def _check(rc: int) -> None:
    if rc != 0:
        raise RuntimeError("trsm oracle: " + ERRORS.get(rc, "error %d" % rc))


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _prep(L, B):
    L = np.ascontiguousarray(L, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.float32)
    if L.ndim != 2 or L.shape[0] != L.shape[1] or B.ndim != 2 or B.shape[0] != L.shape[0]:
        raise ValueError("L must be [n][n] and B [n][m]")
    return L, B


def block_trsm(L, B, tile: int, *, mode: str = "collapsed", threads: int = 1):
    """Solve ``L X = B`` tile by tile in the order of the recurrences; returns ``X`` as float64."""
    L, B = _prep(L, B)
    n, m = B.shape
    X = np.empty((n, m), dtype=np.float64)
    rc = lib().cyc_oracle_block_trsm(MODES[mode], ctypes.c_int64(n), ctypes.c_int64(m), ctypes.c_int64(int(tile)), _ptr(L),
                                     _ptr(B), _ptr(X), int(threads))
    _check(rc)
    return X


def residual(L, B, X, cols):
    """fp64 residual ``B - L X`` and its scale ``|B| + |L||X|`` for the listed columns of a float32 candidate ``X``."""
    L, B = _prep(L, B)
    X = np.ascontiguousarray(X, dtype=np.float32)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    n, m = B.shape
    R = np.empty((n, cols.size), dtype=np.float64)
    S = np.empty((n, cols.size), dtype=np.float64)
    rc = lib().cyc_oracle_trsm_residual(ctypes.c_int64(n), ctypes.c_int64(m), _ptr(L), _ptr(B), _ptr(X), _ptr(cols),
                                        ctypes.c_int64(cols.size), _ptr(R), _ptr(S))
    _check(rc)
    return R, S
