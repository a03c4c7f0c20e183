"""Pins for the FlashAttention-2 oracle: the plain definition softmax(Q K^T / sqrt(d)) V evaluated by library routines,
closed forms, invariants of the recurrence -- nothing here comes from the CUDA path."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

from oracle import fa2
from paper_2511_09987_b200 import inputs


def _rand(seed, N, M, d, scale=1.0):
    r = np.random.default_rng(seed)
    return ((scale * r.standard_normal((N, d))).astype(np.float32), (scale * r.standard_normal((M, d))).astype(np.float32),
            r.uniform(-1, 1, (M, d)).astype(np.float32))


def _definition(Q, K, V):
    scipy_special = pytest.importorskip("scipy.special")
    S = Q.astype(np.float64) @ K.astype(np.float64).T / np.sqrt(Q.shape[1])
    return scipy_special.softmax(S, axis=1) @ V.astype(np.float64), S


@pytest.mark.parametrize("tile", [1, 3, 16, 37, 64, 1000])
@pytest.mark.parametrize("shape", [(5, 37, 8), (16, 64, 16), (3, 129, 4)])
def test_equals_the_plain_definition_for_every_tile_size(tile, shape):
    Q, K, V = _rand(sum(shape) + tile, *shape)
    ref, S = _definition(Q, K, V)
    O, m, l, A = fa2.attention(Q, K, V, tile, with_state=True)
    assert np.abs(O - ref).max() <= 1e-13
    # final state: the row maximum of the scaled scores and the sum of exponentials relative to it
    assert np.abs(m - S.max(axis=1)).max() <= 1e-13
    assert np.abs(l - np.exp(S - S.max(axis=1, keepdims=True)).sum(axis=1)).max() <= 1e-12 * l.max()
    P = np.exp(S - S.max(axis=1, keepdims=True))
    assert np.abs(A - (P / P.sum(axis=1, keepdims=True)) @ np.abs(V.astype(np.float64))).max() <= 1e-13


def test_closed_forms():
    r = np.random.default_rng(3)
    V = r.uniform(-1, 1, (50, 8)).astype(np.float32)
    K = r.standard_normal((50, 8)).astype(np.float32)
    # zero queries: every key weighs the same, the output is the column mean of V
    O = fa2.attention(np.zeros((4, 8), np.float32), K, V, 7)
    assert np.abs(O - V.astype(np.float64).mean(axis=0)).max() <= 1e-15
    # identical keys: same
    O = fa2.attention(r.standard_normal((4, 8)).astype(np.float32), np.tile(K[:1], (50, 1)), V, 16)
    assert np.abs(O - V.astype(np.float64).mean(axis=0)).max() <= 1e-14
    # a single key: the output is its value row, exactly
    O = fa2.attention(r.standard_normal((4, 8)).astype(np.float32), K[:1], V[:1], 5)
    assert (O == np.tile(V[:1].astype(np.float64), (4, 1))).all()
    # one key with an overwhelming score: exp underflows to zero for the rest, the output is that key's value row
    Q = np.zeros((1, 4), np.float32)
    Q[0, 0] = 64.0
    Kb = np.zeros((9, 4), np.float32)
    Kb[5, 0] = 64.0                      # score 64*64/2 = 2048 against 0 for the others
    Vb = r.uniform(-1, 1, (9, 4)).astype(np.float32)
    for tile in (1, 2, 4, 9):
        assert (fa2.attention(Q, Kb, Vb, tile) == Vb[5].astype(np.float64)).all()
    # two keys, scores differing by ln 3 (alpha = 1/2 at d = 4): weights 3/4 and 1/4
    Q = np.array([[2.0, 0, 0, 0]], np.float32)
    K2 = np.array([[np.log(3.0), 0, 0, 0], [0, 0, 0, 0]], np.float64)
    V2 = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]], np.float32)
    O = fa2.attention(Q, K2.astype(np.float32), V2, 1)
    w = np.exp(float(np.float32(np.log(3.0))))            # the float32-rounded key
    assert abs(O[0, 0] - w / (1 + w)) <= 1e-15 and abs(O[0, 1] - 1 / (1 + w)) <= 1e-15


def test_invariants():
    Q, K, V = _rand(11, 9, 70, 8)
    base = fa2.attention(Q, K, V, 16)
    # a permutation of the keys (with their values) changes only the rounding
    perm = np.random.default_rng(1).permutation(70)
    assert np.abs(fa2.attention(Q, K[perm], V[perm], 16) - base).max() <= 1e-14
    # rows of Q are independent, threads change nothing
    assert (fa2.attention(Q[2:5], K, V, 16) == base[2:5]).all()
    assert (fa2.attention(Q, K, V, 16, threads=4) == base).all()
    # outputs are convex combinations of the value rows
    assert (base <= V.max(axis=0) + 1e-15).all() and (base >= V.min(axis=0) - 1e-15).all()
    # large scores do not overflow: the running maximum keeps every exponent <= 0
    big = fa2.attention(40 * Q, 40 * K, V, 16)
    assert np.isfinite(big).all()
    ref, _ = _definition(40 * Q, 40 * K, V)
    assert np.abs(big - ref).max() <= 1e-12


def test_bf16_bit_patterns_are_widened_exactly():
    w = inputs.AttentionWorkload("p", 1, 6, 20, 8, seed=5)
    Q, K, V = inputs.make_attention_operands(w)
    a = fa2.attention(Q[0], K[0], V[0], 8)
    b = fa2.attention(inputs.bf16_bits_to_f32(Q[0]), inputs.bf16_bits_to_f32(K[0]), inputs.bf16_bits_to_f32(V[0]), 8)
    assert (a == b).all()


# ---------------------------------------------------------------------------- planted mistakes
HERE = os.path.dirname(os.path.abspath(fa2.__file__))
MUTANTS = [
    ("scale_one_over_d", "double alpha = 1.0 / sqrt((double)d);", "double alpha = 1.0 / (double)d;"),
    ("running_maximum_not_carried", "double mh = m;", "double mh = -INFINITY;"),
    ("carry_factor_inverted", "double carry = exp(m - mh);", "double carry = exp(mh - m);"),
    ("normaliser_not_rescaled", "l = carry * l;", "l = l;"),
    ("output_not_rescaled", "o[c] = carry * o[c]; a[c] = carry * a[c];", "a[c] = carry * a[c];"),
    ("exponent_relative_to_the_old_maximum", "double e = exp(S[j - j0] - mh);", "double e = exp(S[j - j0] - (j0 ? m : mh));"),
    ("values_of_the_wrong_key", "const float *v = jb->V + j * d;", "const float *v = jb->V + (j1 - 1 - (j - j0)) * d;"),
    ("no_final_division", "jb->O[i * d + c] = o[c] / l;", "jb->O[i * d + c] = o[c];"),
    ("keys_read_transposed", "s += (double)q[c] * (double)k[c];", "s += (double)q[c] * (double)jb->K[c * (M < d ? M : d) % (M * d) + (j % d)];"),
    ("last_partial_tile_dropped", "int64_t j1 = j0 + T < M ? j0 + T : M;", "int64_t j1 = j0 + T; if (j1 > M) break;"),
]


def _pins():
    return [lambda: test_equals_the_plain_definition_for_every_tile_size(3, (5, 37, 8)),
            lambda: test_equals_the_plain_definition_for_every_tile_size(16, (16, 64, 16)),
            lambda: test_equals_the_plain_definition_for_every_tile_size(1000, (3, 129, 4)),
            test_closed_forms, test_invariants]


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(mutant, tmp_path, monkeypatch):
    name, old, new = mutant
    text = open(os.path.join(HERE, "cyc_oracle_fa2.c")).read()
    assert text.count(old) == 1, "mutation site not found: the oracle source changed, update this test"
    (tmp_path / "m.c").write_text(text.replace(old, new, 1))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", *fa2.CFLAGS, "-o", lib_path, str(tmp_path / "m.c"), "-lm"])
    monkeypatch.setattr(fa2, "_lib", ctypes.CDLL(lib_path))
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
