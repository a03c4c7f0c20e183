"""Pins for the CPU oracle: closed forms, hand-worked IEEE cases, the statement
table of Figure "perPE", invariants, brute force and cross-schedule equality.
None of these needs a GPU."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_09987_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DT_NP = {"f32": np.float32, "bf16": np.uint16, "i8": np.int8}
ALL_MODES = ["literal", "wavefront", "os_cannon", "collapsed", "points"]


def enc(dtype, x):
    """Encode small exactly-representable numbers in the operand type."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f32":
        return x.astype(np.float32)
    if dtype == "bf16":
        h = inputs.f32_to_bf16_bits(x.astype(np.float32))
        assert (inputs.bf16_bits_to_f32(h).astype(np.float64) == x).all(), "not exact in bf16"
        return h
    assert (np.abs(x) <= 127).all() or (x >= -128).all()
    return x.astype(np.int8)


def run(mode, dtype, A, B, **kw):
    if mode == "collapsed":
        return oracle.collapsed(dtype, A, B, **kw)
    if mode == "points":
        M = A.shape[0]
        N = B.shape[0] if kw.get("b_col_major") else B.shape[1]
        ii, jj = np.meshgrid(np.arange(M), np.arange(N), indexing="ij")
        return oracle.points(dtype, A, B, ii.ravel(), jj.ravel(), **kw).reshape(M, N)
    return oracle.walk(mode, dtype, A, B, **kw)


# --------------------------------------------------------------------------
# closed forms of C_ij = sum_k A_ik B_kj  (Section "Dataflow Recurrences")
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("mode", ALL_MODES)
def test_identity_and_permutation(dtype, mode):
    rng = np.random.default_rng(5)
    n = 7
    X = rng.integers(-100, 100, size=(n, n)).astype(np.float64)
    X[0, 1], X[1, 0] = 17, -23  # make sure X is not symmetric
    I = np.eye(n)
    P = np.eye(n)[rng.permutation(n)]
    assert not (P == P.T).all()
    assert (run(mode, dtype, enc(dtype, I), enc(dtype, X)) == X).all()         # A = I  =>  C = B
    assert (run(mode, dtype, enc(dtype, X), enc(dtype, I)) == X).all()         # B = I  =>  C = A
    assert (run(mode, dtype, enc(dtype, P), enc(dtype, X)) == P @ X).all()     # row permutation
    assert (run(mode, dtype, enc(dtype, X), enc(dtype, P)) == X @ P).all()     # column permutation
    # B handed over column-major: the stored array is B^T
    assert (run(mode, dtype, enc(dtype, X), enc(dtype, P.T.copy()), b_col_major=True) == X @ P).all()
    assert (run(mode, dtype, enc(dtype, P), enc(dtype, X.T.copy()), b_col_major=True) == P @ X).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("mode", ALL_MODES)
@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 1), (1, 4, 9), (6, 1, 11), (5, 3, 64)])
def test_all_ones(dtype, mode, shape):
    M, N, K = shape
    C = run(mode, dtype, enc(dtype, np.ones((M, K))), enc(dtype, np.ones((K, N))))
    assert C.shape == (M, N) and (C == K).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("mode", ALL_MODES)
def test_rank_one_outer_product(dtype, mode):
    # A = u 1^T, B = 1 v^T  =>  C_ij = K u_i v_j, exact while below 2^24 / 2^31
    M, N, K = 6, 5, 12
    u = np.array([3, -7, 11, 0, 1, -2], dtype=np.float64)
    v = np.array([5, -1, 9, 2, -13], dtype=np.float64)
    A = np.outer(u, np.ones(K))
    B = np.outer(np.ones(K), v)
    assert (run(mode, dtype, enc(dtype, A), enc(dtype, B)) == K * np.outer(u, v)).all()
    assert (run(mode, dtype, enc(dtype, A), enc(dtype, B.T.copy()), b_col_major=True) == K * np.outer(u, v)).all()


def test_int8_extremes_exact():
    K = 4096
    A = np.full((2, K), -128, dtype=np.int8)
    B = np.full((K, 3), -128, dtype=np.int8)
    assert (oracle.collapsed("i8", A, B) == K * 128 * 128).all()          # 2^26, the largest sum of this K
    B[:, 1] = 127
    assert (oracle.collapsed("i8", A, B)[:, 1] == -K * 128 * 127).all()


def test_bf16_widening_values():
    # C = A I returns the operand values widened to fp32: bf16 is the top half of an fp32 word.
    bits = np.array([[0x3F80, 0xC000, 0x3DCD, 0x0001], [0x7F7F, 0x8000, 0x4049, 0x3F81]], dtype=np.uint16)
    want = np.array([[1.0, -2.0, 0.10009765625, 2.0 ** -133],
                     [(2 - 2.0 ** -7) * 2.0 ** 127, -0.0, 3.140625, 1.0078125]])
    I = enc("bf16", np.eye(4))
    got = oracle.walk("literal", "bf16", bits, I)
    assert (got.astype(np.float64) == want).all()


# --------------------------------------------------------------------------
# brute force on tiny shapes, exact rational arithmetic
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("mode", ALL_MODES)
def test_brute_force_tiny_exact(dtype, mode):
    rng = np.random.default_rng(11)
    for (M, N, K) in [(1, 1, 1), (2, 3, 4), (4, 2, 1), (1, 5, 3), (3, 1, 8), (8, 8, 8), (5, 7, 3)]:
        # small integers: every partial sum is exact in every operand type, so any order agrees
        A = rng.integers(-9, 10, size=(M, K)).astype(np.float64)
        B = rng.integers(-9, 10, size=(K, N)).astype(np.float64)
        want = [[sum(Fraction(A[i, k]) * Fraction(B[k, j]) for k in range(K)) for j in range(N)] for i in range(M)]
        got = run(mode, dtype, enc(dtype, A), enc(dtype, B))
        assert got.shape == (M, N)
        for i, j in itertools.product(range(M), range(N)):
            assert Fraction(float(got[i, j])) == want[i][j]
        got_t = run(mode, dtype, enc(dtype, A), enc(dtype, B.T.copy()), b_col_major=True)
        assert (got_t == got).all()


# --------------------------------------------------------------------------
# hand-worked IEEE cases: increasing k from zero, one or two roundings
# --------------------------------------------------------------------------
def _cases():
    out = []
    with open(os.path.join(GOLDEN, "ieee_order_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, a, b, two, fused = [s.strip() for s in line.split("|")]
            out.append((name, [float.fromhex(x) for x in a.split()], [float.fromhex(x) for x in b.split()],
                        float.fromhex(two), float.fromhex(fused)))
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c[0])
@pytest.mark.parametrize("mode", ALL_MODES)
def test_ieee_order_cases(case, mode):
    name, a, b, two, fused = case
    A = np.array([a], dtype=np.float32)
    B = np.array(b, dtype=np.float32).reshape(-1, 1)
    assert (A.astype(np.float64) == np.array([a])).all()  # the fixture values are exact fp32
    for fma, want in ((False, two), (True, fused)):
        got = run(mode, "f32", A, B, fma=fma)
        assert got.shape == (1, 1)
        assert float(got[0, 0]) == want, (name, fma, float(got[0, 0]).hex())
        assert np.signbit(got[0, 0]) == np.signbit(np.float32(want))


def test_order_cases_are_order_sensitive():
    # the fixture really distinguishes orders: the reversed sequence has another hand-worked value
    name, a, b, two, _ = [c for c in _cases() if c[0] == "absorb_up"][0]
    A = np.array([a[::-1]], dtype=np.float32)
    B = np.array(b[::-1], dtype=np.float32).reshape(-1, 1)
    # -2^24 + 1 = -(2^24 - 1) exactly, + 1 = -(2^24 - 2), + 2^24 = 2
    assert float(oracle.walk("literal", "f32", A, B)[0, 0]) == 2.0 != two


# --------------------------------------------------------------------------
# the nine per-cell programs
# --------------------------------------------------------------------------
def _statement_table():
    rows = {}
    with open(os.path.join(GOLDEN, "perpe_statement_table.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            rows[parts[0]] = [int(x) for x in parts[1:]]
    return rows


@pytest.mark.parametrize("mode", ["literal", "wavefront"])
@pytest.mark.parametrize("grid", [(3, 3), (4, 5), (5, 3)])
def test_nine_cell_programs(mode, grid):
    M, K = grid
    N = 4
    table = _statement_table()
    assert list(table) == oracle.CELL_TYPES
    rng = np.random.default_rng(2)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((K, N)).astype(np.float32)
    _, counts = oracle.walk(mode, "f32", A, B, with_counts=True)
    cells_of_type = {"(0,0)": 1, "(0,k)": K - 2, "(0,k_end)": 1, "(i,0)": M - 2, "(i,k)": (M - 2) * (K - 2),
                     "(i,k_end)": M - 2, "(i_end,0)": 1, "(i_end,k)": K - 2, "(i_end,k_end)": 1}
    for t, name in enumerate(oracle.CELL_TYPES):
        per_step = table[name]
        n = cells_of_type[name]
        want = [per_step[0] * n] + [x * n * N for x in per_step[1:]]
        assert counts[t].tolist() == want, (name, counts[t].tolist(), want)
    # I/O summary: A loaded once per cell, B loaded only on the north edge, C written only on the east edge
    assert counts[:, oracle.STATEMENTS.index("load_W")].sum() == M * K
    assert counts[:, oracle.STATEMENTS.index("inject_B")].sum() == K * N
    assert counts[:, oracle.STATEMENTS.index("export_C")].sum() == M * N
    assert counts[:, oracle.STATEMENTS.index("mac")].sum() == M * N * K


# --------------------------------------------------------------------------
# schedules of the same base recurrence agree bit for bit
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("fma", [False, True])
@pytest.mark.parametrize("b_col_major", [False, True])
def test_modes_agree(dtype, fma, b_col_major):
    for n, (M, N, K) in enumerate([(9, 7, 13), (1, 1, 5), (16, 3, 2), (2, 17, 33)]):
        w = inputs.Workload("t", dtype, M, N, K, seed=100 + n, b_col_major=b_col_major,
                            a_dist=("int8",) if dtype == "i8" else ("uniform", -1.0, 1.0),
                            b_dist=("int8",) if dtype == "i8" else ("normal", 1.0))
        A, B = inputs.make_operands(w)
        ref = run("literal", dtype, A, B, fma=fma, b_col_major=b_col_major)
        for mode in ALL_MODES[1:]:
            got = run(mode, dtype, A, B, fma=fma, b_col_major=b_col_major)
            assert got.dtype == ref.dtype and got.tobytes() == ref.tobytes(), mode
        assert oracle.collapsed(dtype, A, B, fma=fma, b_col_major=b_col_major, threads=3).tobytes() == ref.tobytes()
        rows = [M - 1, 0]
        sub = oracle.collapsed(dtype, A, B, fma=fma, b_col_major=b_col_major, rows=rows)
        assert sub.tobytes() == ref[rows].tobytes()


def test_fp32_two_roundings_and_fused_differ_but_are_close():
    A, B = inputs.make_operands(inputs.WORKLOADS["c1"])
    c0 = oracle.collapsed("f32", A, B, fma=False)
    c1 = oracle.collapsed("f32", A, B, fma=True)
    S, _ = oracle.abs_sum_rows("f32", A, B)
    assert (c0 != c1).any()
    assert (np.abs(c0.astype(np.float64) - c1) <= 64 * 2.0 ** -24 * S).all()


def test_bf16_products_are_exact_so_variants_coincide():
    w = inputs.scaled(inputs.WORKLOADS["c5"], batch=1, M=33, N=20, K=70)
    A, B = inputs.make_operands(w)
    assert oracle.collapsed("bf16", A, B, fma=False).tobytes() == oracle.collapsed("bf16", A, B, fma=True).tobytes()


# --------------------------------------------------------------------------
# sequential-summation error bound against the exact sum
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,fma", [("f32", False), ("f32", True), ("bf16", False)])
def test_error_bound_vs_double(dtype, fma):
    M, N, K = 24, 40, 300
    w = inputs.Workload("t", dtype, M, N, K, seed=7, a_dist=("uniform", -1.0, 1.0), b_dist=("normal", 0.1))
    A, B = inputs.make_operands(w)
    C = oracle.collapsed(dtype, A, B, fma=fma).astype(np.float64)
    S, R = oracle.abs_sum_rows(dtype, A, B, threads=2)
    assert (np.abs(C - R) <= 1.01 * K * 2.0 ** -24 * S).all()
    # and the helper sums themselves: against numpy in double
    Af = A.astype(np.float64) if dtype == "f32" else inputs.bf16_bits_to_f32(A).astype(np.float64)
    Bf = B.astype(np.float64) if dtype == "f32" else inputs.bf16_bits_to_f32(B).astype(np.float64)
    assert np.allclose(R, Af @ Bf, rtol=1e-12, atol=1e-12)
    assert np.allclose(S, np.abs(Af) @ np.abs(Bf), rtol=1e-12)
    ii = np.array([0, 5, M - 1])
    jj = np.array([N - 1, 2, 0])
    Sp, Rp = oracle.abs_sum_points(dtype, A, B, ii, jj)
    assert (Sp == S[ii, jj]).all() and (Rp == R[ii, jj]).all()


def test_int8_matches_integer_matmul():
    w = inputs.scaled(inputs.WORKLOADS["c2"], M=37, N=29, K=515)
    A, B = inputs.make_operands(w)
    assert B.shape == (29, 515)
    want = A.astype(np.int64) @ B.astype(np.int64).T
    assert (oracle.collapsed("i8", A, B, b_col_major=True, threads=2) == want).all()


def test_batched_is_independent_problems():
    w = inputs.scaled(inputs.WORKLOADS["c5"], batch=3, M=8, N=9, K=10)
    A, B = inputs.make_operands(w)
    C = oracle.batched_collapsed("bf16", A, B)
    assert C.shape == (3, 8, 9)
    for b in range(3):
        assert (C[b] == oracle.walk("literal", "bf16", A[b], B[b])).all()


def test_bad_arguments_are_rejected():
    A = np.zeros((2, 3), np.float32)
    B = np.zeros((4, 2), np.float32)
    with pytest.raises(ValueError):
        oracle.walk("literal", "f32", A, B)
    with pytest.raises(RuntimeError):
        oracle.points("f32", A, np.zeros((3, 2), np.float32), [2], [0])
    with pytest.raises(RuntimeError):
        oracle.collapsed("f32", A, np.zeros((3, 2), np.float32), rows=[5])
