"""CPU oracle for the Cholesky recurrences (scalar form of Figure "Representative recurrences"; tiled SYRK / GEMM / TRSM /
CHOL form of Section "Simulated Cholesky and Flash Attention").

TEST INFRASTRUCTURE ONLY.  Written in C (``cyc_oracle_chol.c``, fp64) and called through ctypes with numpy arrays.  It
shares nothing with the CUDA library and must not be imported by the product package.

``A`` is ``[n][n]`` float32, symmetric positive definite; only the lower triangle is read.  The factor is ``[n][n]``
float64, lower triangular, ``A = L L^T``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcyc_oracle_chol.so")
_SOURCE = os.path.join(_HERE, "cyc_oracle_chol.c")
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-pthread"]
MODES = {"scalar": 0, "tiled": 1}
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


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(rc):
    if rc:
        raise RuntimeError("cholesky oracle: " + ERRORS.get(rc, "error %d" % rc))


def cholesky(A, tile: int = 0, *, mode: str = "tiled", threads: int = 1):
    """Lower Cholesky factor of ``A`` as float64: ``mode="scalar"`` walks the scalar recurrence entry by entry,
    ``mode="tiled"`` the tiled recurrence with tiles of edge ``tile``."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    if A.ndim != 2 or A.shape[0] != A.shape[1] or A.shape[0] < 1:
        raise ValueError("A must be [n][n]")
    n = A.shape[0]
    L = np.empty((n, n), dtype=np.float64)
    i64 = ctypes.c_int64
    _check(lib().cyc_oracle_cholesky(MODES[mode], i64(n), i64(int(tile) if mode == "tiled" else 1), _ptr(A), _ptr(L), int(threads)))
    return L


def residual(A, L, rows):
    """fp64 residual ``A - L L^T`` and its scale ``|L||L|^T`` on the listed rows (lower triangle) of a float32 candidate ``L``."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    L = np.ascontiguousarray(L, dtype=np.float32)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    n = A.shape[0]
    R = np.empty((len(rows), n), dtype=np.float64)
    S = np.empty((len(rows), n), dtype=np.float64)
    i64 = ctypes.c_int64
    _check(lib().cyc_oracle_cholesky_residual(i64(n), _ptr(A), _ptr(L), _ptr(rows), i64(len(rows)), _ptr(R), _ptr(S)))
    return R, S
