"""CPU oracle for the weight-stationary matrix-multiply recurrence.

TEST INFRASTRUCTURE ONLY.  A plain, slow, literal evaluator of the per-cell
programs of Figure "perPE" and the weight-stationary program of Section
"Space-time Mappings of Dataflow Recurrences", written in C (``cyc_oracle.c``)
and called through ctypes with numpy arrays.  It shares nothing with the CUDA
library and must not be imported by the product package.

Operand conventions: ``A`` is ``[M][K]`` row-major; ``B`` is ``[K][N]``
row-major or, with ``b_col_major=True``, stored as ``[N][K]``; the result is
``[M][N]`` row-major.  dtypes: ``"f32"`` (float32 arrays), ``"bf16"`` (uint16
arrays holding bf16 bit patterns, float32 result) and ``"i8"`` (int8 arrays,
int32 result).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcyc_oracle.so")
_SOURCES = [os.path.join(_HERE, "cyc_oracle.c"), os.path.join(_HERE, "cyc_oracle_walkers.inc")]
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-pthread"]

DTYPES = {"f32": 0, "bf16": 1, "i8": 2}
_IN_NP = {"f32": np.float32, "bf16": np.uint16, "i8": np.int8}
_OUT_NP = {"f32": np.float32, "bf16": np.float32, "i8": np.int32}
MODES = {"literal": 0, "wavefront": 1, "os_cannon": 2}
ERRORS = {1: "bad argument", 2: "out of memory", 3: "copy invariant (i,j,k)_B == B_kj violated",
          4: "channel error: receive without send, or unconsumed send", 5: "timing invariant t = i+j+k violated"}
STATEMENTS = ["load_W", "inject_B", "recv_B", "zero_C", "recv_C", "mac", "send_B", "send_C", "export_C"]
CELL_TYPES = ["(0,0)", "(0,k)", "(0,k_end)", "(i,0)", "(i,k)", "(i,k_end)", "(i_end,0)", "(i_end,k)", "(i_end,k_end)"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SOURCES)
    if stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SOURCES[0], "-lm"], cwd=_HERE)
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
        raise RuntimeError("oracle: " + ERRORS.get(rc, "error %d" % rc))


def _prep(dtype: str, A, B, b_col_major: bool):
    if dtype not in DTYPES:
        raise ValueError("unknown dtype %r" % (dtype,))
    A = np.ascontiguousarray(A, dtype=_IN_NP[dtype])
    B = np.ascontiguousarray(B, dtype=_IN_NP[dtype])
    if A.ndim != 2 or B.ndim != 2:
        raise ValueError("A and B must be matrices")
    M, K = A.shape
    if b_col_major:
        N, K2 = B.shape
    else:
        K2, N = B.shape
    if K2 != K:
        raise ValueError("inner dimensions differ")
    return A, B, M, N, K


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(x):
    return ctypes.c_int64(int(x))


def walk(mode: str, dtype: str, A, B, *, b_col_major: bool = False, fma: bool = False, with_counts: bool = False):
    """Run the ``literal``, ``wavefront`` or ``os_cannon`` walker (small shapes).

    Returns ``C`` or ``(C, counts)``, ``counts[cell_type][statement]`` being how
    often each statement of each of the nine per-cell programs executed.
    """
    A, B, M, N, K = _prep(dtype, A, B, b_col_major)
    C = np.empty((M, N), dtype=_OUT_NP[dtype])
    counts = np.zeros((9, len(STATEMENTS)), dtype=np.int64)
    assert lib().cyc_oracle_statement_count() == len(STATEMENTS)
    rc = lib().cyc_oracle_walk(MODES[mode], DTYPES[dtype], _i64(M), _i64(N), _i64(K), _ptr(A), _ptr(B),
                               int(b_col_major), _ptr(C), int(fma), _ptr(counts) if mode != "os_cannon" else None)
    _check(rc)
    return (C, counts) if with_counts else C


def collapsed(dtype: str, A, B, *, b_col_major: bool = False, fma: bool = False, rows=None, threads: int = 1):
    """Collapsed walker for all rows of C, or for the listed ``rows`` (result ``[len(rows)][N]``)."""
    A, B, M, N, K = _prep(dtype, A, B, b_col_major)
    if rows is None:
        rows_arr, nrows, rows_ptr = None, M, None
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows, rows_ptr = rows_arr.size, _ptr(rows_arr)
    C = np.empty((nrows, N), dtype=_OUT_NP[dtype])
    rc = lib().cyc_oracle_collapsed_rows(DTYPES[dtype], _i64(M), _i64(N), _i64(K), _ptr(A), _ptr(B), int(b_col_major),
                                         rows_ptr, _i64(nrows), _ptr(C), int(fma), int(threads))
    _check(rc)
    return C


def points(dtype: str, A, B, ii, jj, *, b_col_major: bool = False, fma: bool = False):
    """(i,j,k_end)_C for the listed outputs, by the explicit-reduction recurrence."""
    A, B, M, N, K = _prep(dtype, A, B, b_col_major)
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    out = np.empty(ii.size, dtype=_OUT_NP[dtype])
    rc = lib().cyc_oracle_points(DTYPES[dtype], _i64(M), _i64(N), _i64(K), _ptr(A), _ptr(B), int(b_col_major),
                                 _ptr(ii), _ptr(jj), _i64(ii.size), _ptr(out), int(fma))
    _check(rc)
    return out


def abs_sum_points(dtype: str, A, B, ii, jj, *, b_col_major: bool = False):
    """``S = sum_k |A_ik||B_kj|`` and the double-precision sum ``R`` for the listed outputs."""
    A, B, M, N, K = _prep(dtype, A, B, b_col_major)
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    S = np.empty(ii.size, dtype=np.float64)
    R = np.empty(ii.size, dtype=np.float64)
    rc = lib().cyc_oracle_abs_sum_points(DTYPES[dtype], _i64(M), _i64(N), _i64(K), _ptr(A), _ptr(B), int(b_col_major),
                                         _ptr(ii), _ptr(jj), _i64(ii.size), _ptr(S), _ptr(R))
    _check(rc)
    return S, R


def abs_sum_rows(dtype: str, A, B, *, b_col_major: bool = False, rows=None, threads: int = 1):
    """``S`` and ``R`` (see :func:`abs_sum_points`) for all rows or the listed rows."""
    A, B, M, N, K = _prep(dtype, A, B, b_col_major)
    if rows is None:
        nrows, rows_ptr, rows_arr = M, None, None
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows, rows_ptr = rows_arr.size, _ptr(rows_arr)
    S = np.empty((nrows, N), dtype=np.float64)
    R = np.empty((nrows, N), dtype=np.float64)
    rc = lib().cyc_oracle_abs_sum_rows(DTYPES[dtype], _i64(M), _i64(N), _i64(K), _ptr(A), _ptr(B), int(b_col_major),
                                       rows_ptr, _i64(nrows), _ptr(S), _ptr(R), int(threads))
    _check(rc)
    return S, R


def batched_collapsed(dtype: str, A, B, *, b_col_major: bool = False, fma: bool = False, threads: int = 1):
    """Independent recurrences ``A[b] , B[b] -> C[b]`` (leading batch axis), one after another."""
    return np.stack([collapsed(dtype, A[b], B[b], b_col_major=b_col_major, fma=fma, threads=threads)
                     for b in range(len(A))])
