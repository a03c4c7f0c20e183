"""Pins for the block triangular-solve oracle: closed forms, exact integer and rational cases, a library routine on a
special case, invariants of the recurrences (Figure "deps-tri-solve") -- nothing here comes from the CUDA path."""
import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest

from oracle import trsm
from paper_2511_09987_b200 import inputs

ALL_MODES = ["literal", "collapsed"]


def _rng(seed):
    return np.random.default_rng(seed)


def _small_int_system(seed, n, m, unit=True):
    """Integer L (lower), integer X; B = L X computed with Python integers."""
    r = _rng(seed)
    L = np.tril(r.integers(-2, 3, size=(n, n))).astype(np.int64)
    d = np.ones(n, dtype=np.int64) if unit else 2 ** r.integers(0, 3, size=n) * r.choice([-1, 1], size=n)
    L[np.arange(n), np.arange(n)] = d
    X = r.integers(-3, 4, size=(n, m)).astype(np.int64)
    B = np.array([[sum(int(L[i, k]) * int(X[k, j]) for k in range(i + 1)) for j in range(m)] for i in range(n)], dtype=np.int64)
    return L, X, B


@pytest.mark.parametrize("mode", ALL_MODES)
@pytest.mark.parametrize("tile", [1, 2, 3, 5, 64])
def test_identity_and_diagonal(mode, tile):
    r = _rng(1)
    B = r.standard_normal((7, 4)).astype(np.float32)
    assert (trsm.block_trsm(np.eye(7, dtype=np.float32), B, tile, mode=mode) == B.astype(np.float64)).all()
    d = np.array([2.0, -4.0, 0.5, 8.0, -0.25, 1.0, 16.0], dtype=np.float32)
    X = trsm.block_trsm(np.diag(d), B, tile, mode=mode)
    assert (X == B.astype(np.float64) / d.astype(np.float64)[:, None]).all()


@pytest.mark.parametrize("mode", ALL_MODES)
@pytest.mark.parametrize("tile", [1, 3, 4, 11, 32])
@pytest.mark.parametrize("unit", [True, False])
def test_integer_systems_are_solved_exactly(mode, tile, unit):
    # every intermediate value is a small integer (or an integer over a power of two): fp64 is exact
    L, X, B = _small_int_system(7 + tile, 11, 3, unit)
    got = trsm.block_trsm(L.astype(np.float32), B.astype(np.float32), tile, mode=mode)
    assert (got == X.astype(np.float64)).all()


@pytest.mark.parametrize("mode", ALL_MODES)
def test_bidiagonal_closed_form(mode):
    # L = I + a * subdiagonal, B = e_0  =>  X_i = (-a)^i
    n, a = 40, 0.5
    L = np.eye(n, dtype=np.float32) + a * np.eye(n, k=-1, dtype=np.float32)
    B = np.zeros((n, 1), dtype=np.float32)
    B[0, 0] = 1.0
    X = trsm.block_trsm(L, B, 8, mode=mode)
    assert (X[:, 0] == np.array([(-a) ** i for i in range(n)])).all()


@pytest.mark.parametrize("mode", ALL_MODES)
def test_all_ones_lower_triangle(mode):
    # L = lower triangle of ones: X_0 = B_0, X_i = B_i - B_{i-1}
    n = 23
    B = np.arange(1, n + 1, dtype=np.float32)[:, None] ** 2 * np.array([[1.0, -2.0]], dtype=np.float32)
    X = trsm.block_trsm(np.tril(np.ones((n, n), dtype=np.float32)), B, 4, mode=mode)
    want = np.vstack([B[:1], B[1:] - B[:-1]]).astype(np.float64)
    assert (X == want).all()


@pytest.mark.parametrize("mode", ALL_MODES)
@pytest.mark.parametrize("shape", [(1, 1, 1), (2, 1, 1), (6, 2, 4), (9, 3, 4), (8, 2, 8)])
def test_exact_rational_substitution(mode, shape):
    n, m, tile = shape
    r = _rng(n * 100 + m)
    L = (r.integers(-8, 9, size=(n, n)) / 8.0).astype(np.float32)
    L[np.arange(n), np.arange(n)] = (r.integers(8, 17, size=n) / 8.0 * r.choice([-1, 1], size=n)).astype(np.float32)
    B = (r.integers(-16, 17, size=(n, m)) / 4.0).astype(np.float32)
    exact = [[None] * m for _ in range(n)]
    for j in range(m):
        for i in range(n):
            s = Fraction(float(B[i, j]))
            for k in range(i):
                s -= Fraction(float(L[i, k])) * exact[k][j]
            exact[i][j] = s / Fraction(float(L[i, i]))
    X = trsm.block_trsm(L, B, tile, mode=mode)
    for i in range(n):
        for j in range(m):
            e = float(exact[i][j])
            assert abs(X[i, j] - e) <= 1e-13 * max(1.0, abs(e)), (i, j)


@pytest.mark.parametrize("coupling", ["dominant", "sqrt"])
def test_library_triangular_solve(coupling):
    scipy_linalg = pytest.importorskip("scipy.linalg")
    w = inputs.TrsmWorkload("p", 97, 5, 16, seed=3, coupling=coupling)
    L, B = inputs.make_trsm_operands(w)
    X = trsm.block_trsm(L, B, w.tile)
    ref = scipy_linalg.solve_triangular(np.tril(L).astype(np.float64), B.astype(np.float64), lower=True)
    assert np.abs(X - ref).max() <= 1e-12 * np.abs(ref).max()


def test_modes_agree_bit_for_bit_and_tile_size_only_moves_roundings():
    w = inputs.TrsmWorkload("p", 45, 7, 8, seed=5, coupling="sqrt")
    L, B = inputs.make_trsm_operands(w)
    base = trsm.block_trsm(L, B, 8, mode="collapsed")
    assert (trsm.block_trsm(L, B, 8, mode="literal") == base).all()
    assert (trsm.block_trsm(L, B, 8, mode="collapsed", threads=3) == base).all()
    for tile in (1, 3, 45, 64):
        other = trsm.block_trsm(L, B, tile, mode="literal")
        assert (trsm.block_trsm(L, B, tile, mode="collapsed") == other).all()
        assert np.abs(other - base).max() <= 1e-13 * np.abs(base).max()


def test_upper_triangle_is_never_read_and_columns_are_independent():
    w = inputs.TrsmWorkload("p", 33, 6, 8, seed=6)
    L, B = inputs.make_trsm_operands(w)
    assert np.isnan(L[0, 1])
    X = trsm.block_trsm(L, B, 8)
    assert np.isfinite(X).all()
    L2 = L.copy()
    L2[np.triu_indices(33, 1)] = 7.0
    assert (trsm.block_trsm(L2, B, 8) == X).all()
    assert (trsm.block_trsm(L, B[:, 2:4], 8) == X[:, 2:4]).all()


@pytest.mark.parametrize("coupling", ["dominant", "sqrt"])
def test_residual_of_the_solution_is_at_rounding_level(coupling):
    w = inputs.TrsmWorkload("p", 200, 9, 32, seed=8, coupling=coupling)
    L, B = inputs.make_trsm_operands(w)
    X = trsm.block_trsm(L, B, w.tile, threads=2)
    L64 = np.tril(L).astype(np.float64)
    R = B.astype(np.float64) - L64 @ X
    S = np.abs(B.astype(np.float64)) + np.abs(L64) @ np.abs(X)
    assert (np.abs(R) <= 200 * 2.0 ** -52 * S).all()
    # the residual helper agrees with this numpy evaluation on an fp32 candidate
    cols = np.array([0, 4, 8])
    Xc = X.astype(np.float32)
    R2, S2 = trsm.residual(L, B, Xc, cols)
    R3 = B.astype(np.float64)[:, cols] - L64 @ Xc.astype(np.float64)[:, cols]
    assert np.abs(R2 - R3).max() <= 1e-12
    assert np.abs(S2 - (np.abs(B.astype(np.float64)) + np.abs(L64) @ np.abs(Xc.astype(np.float64)))[:, cols]).max() <= 1e-12


def test_dominant_generator_keeps_its_promise():
    w = inputs.TrsmWorkload("p", 300, 2, 32, seed=9)
    L, _ = inputs.make_trsm_operands(w)
    off = np.abs(np.tril(L, -1).astype(np.float64)).sum(axis=1)
    d = np.abs(np.diag(L))
    assert off.max() < 0.5 and d.min() >= 1.0 and d.max() < 2.0
    assert (np.diag(L) < 0).any() and (np.diag(L) > 0).any()


# ---------------------------------------------------------------------------- planted mistakes
HERE = os.path.dirname(os.path.abspath(trsm.__file__))
MUTANTS = [
    ("gemm_update_added_to_the_right_hand_side", "rhs[r * m + c] = (double)B[(r0 + r) * m + c] - xa;", "rhs[r * m + c] = (double)B[(r0 + r) * m + c] + xa;"),
    ("collapsed_update_added", "xa[c] = (double)jb->B[r * m + c0 + c] - xa[c]; /* B_i - Xa */", "xa[c] = (double)jb->B[r * m + c0 + c] + xa[c];"),
    ("substitution_reads_l_transposed", "double p = (double)L[(r0 + r) * n + (r0 + k)] * X[k * w + c];", "double p = (double)L[(r0 + k) * n + (r0 + r)] * X[k * w + c];"),
    ("substitution_skips_first_column_of_the_tile", "for (int64_t k = 0; k < r; ++k) {\n                double p = (double)L[(r0 + r)", "for (int64_t k = 1; k < r; ++k) {\n                double p = (double)L[(r0 + r)"),
    ("multiplies_by_the_diagonal", "X[r * w + c] = s / d;", "X[r * w + c] = s * d;"),
    ("collapsed_multiplies_by_the_diagonal", "Xr[c] = xa[c] / d;", "Xr[c] = xa[c] * d;"),
    ("first_block_column_dropped", "tile_gemm(L, n, r0, rows_i, k0, rows_j, xb, xa, m);\n        }", "if (j > 0) tile_gemm(L, n, r0, rows_i, k0, rows_j, xb, xa, m);\n        }"),
    ("collapsed_drops_the_last_row_of_each_earlier_block", "for (int64_t k = 0; k < r0; ++k) { /* blocks j = 0..i-1, k increasing */", "for (int64_t k = 0; k < r0 - 1; ++k) { /* planted */"),
    ("accumulator_not_zeroed_at_west_boundary", "if (j == 0) for (int64_t e = 0; e < rows_i * m; ++e) xa[e] = 0.0;", "if (j == 0) for (int64_t e = 0; e < rows_i * m; ++e) xa[e] = 1.0;"),
    ("seed_taken_from_the_wrong_diagonal_point", "const double *from = (i == j + 1) ? Xd[j] : Xb[(i - 1) * nb + j];", "const double *from = (i == j + 1) ? Xd[0] : Xb[(i - 1) * nb + j];"),
    ("gemm_reads_l_from_the_diagonal_tile", "double l = (double)L[(r0 + r) * n + (k0 + k)];", "double l = (double)L[(r0 + r) * n + (r0 + k)];"),
]


def _pins():
    out = []
    for mode in ALL_MODES:
        out.append(lambda m=mode: test_identity_and_diagonal(m, 3))
        out.append(lambda m=mode: test_integer_systems_are_solved_exactly(m, 4, True))
        out.append(lambda m=mode: test_integer_systems_are_solved_exactly(m, 3, False))
        out.append(lambda m=mode: test_bidiagonal_closed_form(m))
        out.append(lambda m=mode: test_all_ones_lower_triangle(m))
        out.append(lambda m=mode: test_exact_rational_substitution(m, (9, 3, 4)))
    out.append(test_modes_agree_bit_for_bit_and_tile_size_only_moves_roundings)
    out.append(lambda: test_library_triangular_solve("sqrt"))
    return out


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(mutant, tmp_path, monkeypatch):
    name, old, new = mutant
    text = open(os.path.join(HERE, "cyc_oracle_trsm.c")).read()
    assert text.count(old) == 1, "mutation site not found: the oracle source changed, update this test"
    (tmp_path / "m.c").write_text(text.replace(old, new, 1))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", *trsm.CFLAGS, "-o", lib_path, str(tmp_path / "m.c"), "-lm"])
    monkeypatch.setattr(trsm, "_lib", ctypes.CDLL(lib_path))
    caught = 0
    for pin in _pins():
        try:
            pin()
        except (AssertionError, RuntimeError, OverflowError, ValueError, ZeroDivisionError):
            caught += 1
    assert caught > 0, "no pin noticed the planted mistake %r" % name


def test_unmodified_oracle_passes_the_same_pins():
    for pin in _pins():
        pin()
