"""Pins for the Cholesky oracle (scalar recurrence of Figure "Representative recurrences", tiled SYRK / GEMM / TRSM / CHOL
recurrence of Section "Simulated Cholesky and Flash Attention"): closed forms, exact integer and rational cases, a library
factorisation, invariants -- nothing here comes from the CUDA path."""
import ctypes
import os
import subprocess
from fractions import Fraction
from math import comb

import numpy as np
import pytest

from oracle import chol

TILES = [1, 2, 3, 5, 8, 64]


def both(A, tile):
    a = chol.cholesky(A, mode="scalar")
    b = chol.cholesky(A, tile, mode="tiled")
    assert a.tobytes() == b.tobytes(), "scalar and tiled walks disagree"
    return b


def _spd(seed, n):
    r = np.random.default_rng(seed)
    M = r.standard_normal((n, n))
    return (M @ M.T / n + np.eye(n)).astype(np.float32)


@pytest.mark.parametrize("tile", TILES)
def test_closed_forms(tile):
    n = 11
    assert (both(np.eye(n, dtype=np.float32), tile) == np.eye(n)).all()
    d = np.array([4.0, 9.0, 0.25, 16.0, 1.0, 2.25, 64.0], dtype=np.float32)
    assert (both(np.diag(d), tile) == np.diag(np.sqrt(d.astype(np.float64)))).all()
    # A_ij = min(i, j) + 1: the factor is the all-ones lower triangle
    i = np.arange(n)
    assert (both((np.minimum.outer(i, i) + 1).astype(np.float32), tile) == np.tril(np.ones((n, n)))).all()
    # Pascal matrix C(i+j, i): the factor holds the binomial coefficients C(i, j), exactly
    P = np.array([[comb(a + b, a) for b in range(n)] for a in range(n)], dtype=np.float32)
    want = np.array([[comb(a, b) if b <= a else 0 for b in range(n)] for a in range(n)], dtype=np.float64)
    assert (both(P, tile) == want).all()
    # A_ij = rho^|i-j| (rho = 1/2): L_i0 = rho^i, L_ij = rho^(i-j) sqrt(1 - rho^2)
    rho = 0.5
    A = (rho ** np.abs(np.subtract.outer(i, i))).astype(np.float32)
    want = np.tril(rho ** np.subtract.outer(i, i).clip(0).astype(np.float64)) * np.sqrt(1 - rho * rho)
    want[:, 0] = rho ** i
    assert np.abs(both(A, tile) - want).max() <= 4e-16
    # 1 x 1 and 2 x 2 by hand: [[4, 2], [2, 10]] = [[2, 0], [1, 3]] [[2, 1], [0, 3]]
    assert both(np.array([[9.0]], dtype=np.float32), tile).tolist() == [[3.0]]
    assert both(np.array([[4.0, 2.0], [2.0, 10.0]], dtype=np.float32), tile).tolist() == [[2.0, 0.0], [1.0, 3.0]]


@pytest.mark.parametrize("tile", TILES)
def test_integer_factor_is_recovered_exactly(tile):
    r = np.random.default_rng(4)
    n = 13
    L0 = np.tril(r.integers(-3, 4, size=(n, n))).astype(np.int64)
    L0[np.arange(n), np.arange(n)] = r.integers(1, 5, size=n)            # positive diagonal: the factor is unique
    A = np.array([[sum(int(L0[a, k]) * int(L0[b, k]) for k in range(n)) for b in range(n)] for a in range(n)])
    assert (both(A.astype(np.float32), tile) == L0).all()


def test_exact_rational_reconstruction_and_library():
    for seed, n in ((1, 6), (2, 9)):
        A = _spd(seed, n)
        L = both(A, 4)
        for a in range(n):
            for b in range(a + 1):
                acc = sum(Fraction(float(L[a, k])) * Fraction(float(L[b, k])) for k in range(b + 1))
                scale = sum(abs(Fraction(float(L[a, k])) * Fraction(float(L[b, k]))) for k in range(b + 1))
                assert abs(Fraction(float(A[a, b])) - acc) <= (n + 2) * Fraction(2) ** -52 * scale
    A = _spd(7, 97)
    assert np.abs(both(A, 16) - np.linalg.cholesky(A.astype(np.float64))).max() <= 1e-13


def test_invariants():
    A = _spd(3, 40)
    L = both(A, 8)
    assert (np.triu(L, 1) == 0).all() and (np.diag(L) > 0).all()
    # only the lower triangle of A is read
    B = A.copy()
    B[np.triu_indices(40, 1)] = np.nan
    assert chol.cholesky(B, 8).tobytes() == L.tobytes()
    assert chol.cholesky(B, mode="scalar").tobytes() == L.tobytes()
    # threads change nothing
    assert chol.cholesky(A, 8, threads=5).tobytes() == L.tobytes()
    # the leading principal block has the leading block of L as its factor
    assert chol.cholesky(A[:17, :17], 8).tobytes() == np.ascontiguousarray(L[:17, :17]).tobytes()
    # scaling A by 4 scales L by 2, exactly
    assert (chol.cholesky(4 * A, 8) == 2 * L).all()
    # D A D with D = diag of powers of two scales the rows of L, exactly
    dd = 2.0 ** np.random.default_rng(0).integers(-2, 3, size=40)
    assert (chol.cholesky((dd[:, None] * A * dd[None, :]).astype(np.float32), 8) == dd[:, None] * L).all()
    # not positive definite: the square root of a negative pivot is NaN, not an error
    bad = chol.cholesky(np.array([[1.0, 2.0], [2.0, 1.0]], dtype=np.float32), 1)
    assert bad[0, 0] == 1.0 and bad[1, 0] == 2.0 and np.isnan(bad[1, 1])


def test_residual_helper():
    A = _spd(5, 30)
    L = chol.cholesky(A, 8).astype(np.float32)
    rows = np.array([0, 7, 29])
    R, S = chol.residual(A, L, rows)
    L64 = L.astype(np.float64)
    want = (A.astype(np.float64) - L64 @ L64.T)[rows]
    scale = (np.abs(L64) @ np.abs(L64).T)[rows]
    for q, i in enumerate(rows):
        assert np.abs(R[q, :i + 1] - want[q, :i + 1]).max() <= 1e-14
        assert np.abs(S[q, :i + 1] - scale[q, :i + 1]).max() <= 1e-13
        assert (R[q, i + 1:] == 0).all() and (S[q, i + 1:] == 0).all()
    assert np.abs(R).max() <= 30 * 2.0 ** -24 * S.max()   # fp32-rounded factor: residual at fp32 rounding level


# ---------------------------------------------------------------------------- planted mistakes
HERE = os.path.dirname(os.path.abspath(chol.__file__))
MUTANTS = [
    ("scalar_diagonal_without_sqrt", "if (i == j) L[i * n + i] = sqrt(s);", "if (i == j) L[i * n + i] = s;"),
    ("scalar_divides_by_the_wrong_pivot", "else L[i * n + j] = s / L[j * n + j];", "else L[i * n + j] = s / L[i * n + i - (i > 0)];"),
    ("scalar_update_added", "for (int64_t k = 0; k < j; ++k) s = s - L[i * n + k] * L[j * n + k];\n            if (i == j)",
     "for (int64_t k = 0; k < j; ++k) s = s + L[i * n + k] * L[j * n + k];\n            if (i == j)"),
    ("update_of_one_panel_dropped", "for (int64_t k = 0; k < J; ++k)   /* SYRK", "for (int64_t k = (J > 1); k < J; ++k)   /* SYRK"),
    ("update_uses_the_same_rows_twice", "s = s - L[(r0 + r) * n + k0 + k] * L[(c0 + c) * n + k0 + k];", "s = s - L[(r0 + r) * n + k0 + k] * L[(r0 + c) * n + k0 + k];"),
    ("tile_chol_multiplies_by_the_pivot", "S[i * lds + j] = (i == j) ? sqrt(s) : s / S[j * lds + j];", "S[i * lds + j] = (i == j) ? sqrt(s) : s * S[j * lds + j];"),
    ("trsm_with_untransposed_factor", "s = s - S[r * lds + k] * Ljj[c * ldl + k];", "s = s - S[r * lds + k] * Ljj[k * ldl + c];"),
    ("trsm_without_division", "S[r * lds + c] = s / Ljj[c * ldl + c];", "S[r * lds + c] = s;"),
    ("trsm_uses_the_wrong_diagonal_tile", "tile_trsm_right(L + c0 * n + c0, n, S, rows, cols, cols);", "tile_trsm_right(L + (c0 ? c0 - b : 0) * (n + 1), n, S, rows, cols, cols);"),
    ("upper_triangle_of_A_read", "S[r * cols + c] = (r0 + r >= c0 + c) ? (double)A[(r0 + r) * n + c0 + c] : 0.0;", "S[r * cols + c] = (double)A[(c0 + c) * n + r0 + r];"),
    ("residual_scale_without_abs", "sc = sc + fabs(p);", "sc = sc + p;"),
    ("residual_sums_past_the_diagonal", "for (int64_t k = 0; k <= j; ++k) {\n                    const double p", "for (int64_t k = 0; k < j; ++k) {\n                    const double p"),
]


def _pins():
    return ([(lambda t=t: test_closed_forms(t)) for t in (1, 3, 64)] + [(lambda t=t: test_integer_factor_is_recovered_exactly(t)) for t in (2, 5)]
            + [test_exact_rational_reconstruction_and_library, test_invariants, test_residual_helper])


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(mutant, tmp_path, monkeypatch):
    name, old, new = mutant
    text = open(os.path.join(HERE, "cyc_oracle_chol.c")).read()
    assert text.count(old) == 1, "mutation site not found: the oracle source changed, update this test"
    (tmp_path / "m.c").write_text(text.replace(old, new, 1))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", *chol.CFLAGS, "-o", lib_path, str(tmp_path / "m.c"), "-lm"])
    monkeypatch.setattr(chol, "_lib", ctypes.CDLL(lib_path))
    caught = 0
    for pin in _pins():
        try:
            pin()
        except (AssertionError, RuntimeError, OverflowError, ValueError, ZeroDivisionError, FloatingPointError):
            caught += 1
    assert caught > 0, "no pin noticed the planted mistake %r" % name


def test_unmodified_oracle_passes_the_same_pins():
    for pin in _pins():
        pin()
