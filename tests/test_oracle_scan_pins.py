"""Pins for the prefix-sum oracle (``P_i = P_{i-1} + A_i``, Figure "Representative recurrences"): closed forms, exact
integer arithmetic with Python integers and fractions, hand-worked IEEE-754 cases that fix the order and the start,
invariants, a library routine -- nothing here comes from the CUDA path."""
import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest

from oracle import scan

ARITH = ["f64", "f32", "i32"]


def _ints(seed, n, lo=-1000, hi=1000):
    return np.random.default_rng(seed).integers(lo, hi, size=n)


@pytest.mark.parametrize("arith", ARITH)
def test_closed_forms(arith):
    dt = np.int32 if arith == "i32" else np.float32
    n = 3000
    # all ones: P_i = i + 1
    assert (scan.prefix_sum(np.ones(n, dt), arithmetic=arith) == np.arange(1, n + 1)).all()
    # A_i = i: triangular numbers (exact in fp32 up to 2^24: 3000*2999/2 < 2^23)
    assert (scan.prefix_sum(np.arange(n).astype(dt), arithmetic=arith) == np.arange(n) * (np.arange(n) + 1) // 2).all()
    # alternating signs: 1, 0, 1, 0, ...
    a = np.where(np.arange(n) % 2 == 0, 1, -1).astype(dt)
    assert (scan.prefix_sum(a, arithmetic=arith) == (np.arange(n) + 1) % 2).all()
    # telescoping differences of a known sequence give the sequence back
    p = (np.arange(n) % 97 - 48) * 3
    a = np.diff(p, prepend=0).astype(dt)
    assert (scan.prefix_sum(a, arithmetic=arith) == p).all()
    # a single element, an empty sequence
    assert scan.prefix_sum(np.array([7], dt), arithmetic=arith).tolist() == [7]
    assert scan.prefix_sum(np.zeros(0, dt), arithmetic=arith).shape == (0,)


@pytest.mark.parametrize("arith", ARITH)
def test_exact_against_python_integers(arith):
    a = _ints(3, 4097)
    want, run = [], 0
    for x in a.tolist():
        run += x
        want.append(run)
    got = scan.prefix_sum(a.astype(np.int32 if arith == "i32" else np.float32), arithmetic=arith)
    assert got.tolist() == want


def test_f64_against_exact_rationals_and_scale():
    r = np.random.default_rng(5)
    a = r.standard_normal(600).astype(np.float32)
    P, S = scan.prefix_sum(a, arithmetic="f64", with_scale=True)
    run, runabs = Fraction(0), Fraction(0)
    for i, x in enumerate(a.tolist()):
        run += Fraction(x)
        runabs += abs(Fraction(x))
        assert abs(Fraction(float(P[i])) - run) <= Fraction(2) ** -52 * runabs * (i + 1)
        assert abs(Fraction(float(S[i])) - runabs) <= Fraction(2) ** -52 * runabs * (i + 1)
    # the last element equals a correctly rounded library sum to rounding level
    import math
    assert abs(P[-1] - math.fsum(a.astype(np.float64))) <= 600 * 2.0 ** -52 * float(S[-1])


def test_int32_wraps_around():
    a = np.array([2 ** 31 - 1, 1, 1, -(2 ** 31), 5], dtype=np.int32)
    got = scan.prefix_sum(a, arithmetic="i32").tolist()
    assert got == [2 ** 31 - 1, -(2 ** 31), -(2 ** 31) + 1, 1, 6]
    big = _ints(9, 5000, -2 ** 31, 2 ** 31)
    want = ((np.cumsum(big.astype(object)) + 2 ** 31) % 2 ** 32 - 2 ** 31).astype(np.int64)
    assert (scan.prefix_sum(big.astype(np.int32), arithmetic="i32") == want).all()


def test_f32_order_and_start_hand_worked():
    """Hand-worked IEEE-754 single-precision cases.  2^24 + 1 is not representable: the tie rounds to even (2^24), so
    adding 1 twice to 2^24 one at a time stays at 2^24, whereas any order that first forms 1 + 1 = 2 reaches 2^24 + 2."""
    a = np.array([2.0 ** 24, 1.0, 1.0], dtype=np.float32)
    assert scan.prefix_sum(a, arithmetic="f32").tolist() == [2.0 ** 24, 2.0 ** 24, 2.0 ** 24]
    assert scan.prefix_sum(a, arithmetic="f64").tolist() == [2.0 ** 24, 2.0 ** 24 + 1, 2.0 ** 24 + 2]
    # increasing i, not decreasing: from the other end the small terms would be absorbed differently
    a = np.array([1.0, 1.0, 2.0 ** 24], dtype=np.float32)
    assert scan.prefix_sum(a, arithmetic="f32").tolist() == [1.0, 2.0, 2.0 ** 24 + 2]
    # the start is +0: P_0 = 0 + A_0, so a negative zero input gives +0
    z = scan.prefix_sum(np.array([-0.0], dtype=np.float32), arithmetic="f32")
    assert z[0] == 0.0 and not np.signbit(z[0])
    # cancellation: 1e8 - 1e8 + 1 = 1, element by element
    a = np.array([1e8, -1e8, 1.0], dtype=np.float32)
    assert scan.prefix_sum(a, arithmetic="f32").tolist() == [1e8, 0.0, 1.0]


def test_invariants():
    r = np.random.default_rng(11)
    a = r.uniform(-1, 1, 2000).astype(np.float32)
    P = scan.prefix_sum(a, arithmetic="f64")
    # first differences give A back (to fp64 rounding)
    assert np.abs(np.diff(P, prepend=0.0) - a).max() <= 2000 * 2.0 ** -52
    # P_i depends on A_0..A_i only
    b = a.copy()
    b[1500:] = 99.0
    assert (scan.prefix_sum(b, arithmetic="f64")[:1500] == P[:1500]).all()
    # linearity in fp64 up to rounding; scaling by a power of two is exact
    assert (scan.prefix_sum(a * np.float32(4.0), arithmetic="f64") == 4.0 * P).all()
    assert (scan.prefix_sum(a * np.float32(0.5), arithmetic="f32") == 0.5 * scan.prefix_sum(a, arithmetic="f32")).all()
    # splitting a sequence: the second part continues from the last value of the first
    k = 777
    tail = scan.prefix_sum(a[k:], arithmetic="f64")
    assert np.abs(P[k:] - (P[k - 1] + tail)).max() <= 2000 * 2.0 ** -52
    # the fp32 walk stays within the sequential-summation bound of the fp64 walk
    P32 = scan.prefix_sum(a, arithmetic="f32")
    _, S = scan.prefix_sum(a, arithmetic="f64", with_scale=True)
    assert (np.abs(P32 - P) <= 1.01 * (np.arange(2000) + 1) * 2.0 ** -24 * S).all()
    assert np.abs(P32 - P).max() > 0  # and it is a different arithmetic


def test_rows_are_independent_sequences():
    r = np.random.default_rng(13)
    a = r.integers(-50, 50, size=(5, 311)).astype(np.int32)
    for arith, dt in (("i32", np.int32), ("f32", np.float32), ("f64", np.float32)):
        got = scan.prefix_sum(a.astype(dt), arithmetic=arith)
        for row in range(5):
            assert (got[row] == scan.prefix_sum(a[row].astype(dt), arithmetic=arith)).all()
        assert (got == np.cumsum(a.astype(np.int64), axis=1)).all()  # exact integers: the library's cumulative sum


# ---------------------------------------------------------------------------- planted mistakes
HERE = os.path.dirname(os.path.abspath(scan.__file__))
MUTANTS = [
    ("exclusive_instead_of_inclusive_f64", "prev = prev + a;             /* P_i = P_{i-1} + A_i */\n            P[r * stride + i] = prev;",
     "P[r * stride + i] = prev;\n            prev = prev + a;"),
    ("subtracts_f64", "prev = prev + a;             /* P_i", "prev = prev - a;             /* P_i"),
    ("row_does_not_restart_f64", "        double prev = 0.0;   /* P_{-1} */\n", "        static double prev = 0.0;\n"),
    ("scale_without_abs", "scale = scale + fabs(a);", "scale = scale + a;"),
    ("start_is_not_zero_f32", "volatile float prev = 0.0f;", "volatile float prev = 1.0f;"),
    ("f32_kept_in_double", "volatile float prev = 0.0f;", "double prev = 0.0;"),
    ("reads_the_next_element_i32", "prev = prev + (uint32_t)A[r * stride + i];", "prev = prev + (uint32_t)A[r * stride + (i + 1 < n ? i + 1 : i)];"),
    ("saturates_i32", "P[r * stride + i] = (int32_t)prev;",
     "P[r * stride + i] = (i && ((int32_t)prev < P[r * stride + i - 1]) && A[r * stride + i] > 0) ? INT32_MAX : (int32_t)prev;"),
    ("wrong_row_stride_i32", "uint32_t prev = 0u;\n        for (int64_t i = 0; i < n; ++i) {\n            prev = prev + (uint32_t)A[r * stride + i];",
     "uint32_t prev = 0u;\n        for (int64_t i = 0; i < n; ++i) {\n            prev = prev + (uint32_t)A[(r ? r - 1 : 0) * stride + i];"),
]


def _pins():
    return ([(lambda a=a: test_closed_forms(a)) for a in ARITH] + [(lambda a=a: test_exact_against_python_integers(a)) for a in ARITH]
            + [test_f64_against_exact_rationals_and_scale, test_int32_wraps_around, test_f32_order_and_start_hand_worked,
               test_invariants, test_rows_are_independent_sequences])


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(mutant, tmp_path, monkeypatch):
    name, old, new = mutant
    text = open(os.path.join(HERE, "cyc_oracle_scan.c")).read()
    assert text.count(old) == 1, "mutation site not found: the oracle source changed, update this test"
    (tmp_path / "m.c").write_text(text.replace(old, new, 1))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", *scan.CFLAGS, "-o", lib_path, str(tmp_path / "m.c"), "-lm"])
    monkeypatch.setattr(scan, "_lib", ctypes.CDLL(lib_path))
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
