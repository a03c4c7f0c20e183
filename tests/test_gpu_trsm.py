"""Block lower-triangular solve on the GPU against the fp64 oracle on the same seeded operands.

Acceptance (fp32 arithmetic on the GPU, fp64 in the oracle):
* backward: the residual of the GPU solution satisfies ``|B - L X| <= 1e-5 * (|B| + |L||X|)`` element by element
  (forward substitution is backward stable with a constant of order ``n * 2^-24`` in the worst case and
  ``sqrt(n) * 2^-24`` for random data; 1e-5 is the fp32 tolerance of the matrix-multiply path);
* forward, diagonally dominant ``L`` (``|L^-1|`` bounded by 2 in the infinity norm, so the error of a column is at
  most twice its largest residual): ``|X - X_oracle| <= 2e-5 * max_r (|B| + |L||X|)_r`` per column, element by element;
* forward, order-one coupling: ``|X - X_oracle| <= 1e-4 * max|X_oracle|`` per column (the error growth of this
  generator is bounded by a small constant, measured well below 10).
"""
import numpy as np
import pytest

from oracle import trsm as otrsm
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu
TW = inputs.TrsmWorkload


def gpu_solve(L, B, tile, fixed=False, in_place=False):
    import torch
    from paper_2511_09987_b200 import binding
    dL = torch.from_numpy(L).cuda()
    dB = torch.from_numpy(B).cuda()
    X = binding.block_trsm(dL, dB, dB if in_place else None, tile=tile, fixed_k_order=fixed)
    assert binding.last_device_status() == binding.CYC_OK
    torch.cuda.synchronize()
    if not in_place:
        assert (dB.cpu().numpy() == B).all(), "B was modified"
    return X.cpu().numpy()


def check(w, X, L, B, cols=None, threads=8):
    n, m = B.shape
    cols = np.arange(m) if cols is None else np.asarray(cols)
    assert X.shape == (n, m) and X.dtype == np.float32 and np.isfinite(X).all()
    ref = otrsm.block_trsm(L, np.ascontiguousarray(B[:, cols]), w.tile, threads=threads)
    R, S = otrsm.residual(L, B, X, cols)
    assert (np.abs(R) <= 1e-5 * S).all(), "residual %g of its scale" % float((np.abs(R) / S).max())
    err = np.abs(X[:, cols].astype(np.float64) - ref)
    if w.coupling == "dominant":
        bound = 2e-5 * S.max(axis=0, keepdims=True)
    else:
        bound = 1e-4 * np.abs(ref).max(axis=0, keepdims=True)
    assert (err <= bound).all(), "forward error %g of its bound" % float((err / bound).max())
    return float((np.abs(R) / S).max()), float((err / bound).max())


CASES = [
    TW("one", 1, 1, 1, seed=20),
    TW("tiny_unaligned", 5, 3, 2, seed=21),
    TW("one_tile", 96, 40, 256, seed=22),
    TW("ragged_rows_in_tile", 77, 33, 32, seed=23),
    TW("t1", 512, 96, 64, seed=10),
    TW("odd_everything", 301, 30, 40, seed=24),
    TW("ragged_last_tile", 700, 200, 256, seed=25),
    TW("three_blocks", 700, 200, 96 * 2 + 64, seed=26),
    TW("tensor_core_updates", 1024, 512, 256, seed=27),
    TW("tensor_core_updates_ragged", 1500, 260, 256, seed=28),
    TW("order_one_coupling", 1024, 256, 128, seed=29, coupling="sqrt"),
    TW("many_small_tiles", 256, 64, 8, seed=30, coupling="sqrt"),
]


@pytest.mark.parametrize("w", CASES, ids=[c.name for c in CASES])
@pytest.mark.parametrize("fixed", [False, True], ids=["default", "fixed_k_order"])
def test_against_the_oracle(w, fixed):
    L, B = inputs.make_trsm_operands(w)
    X = gpu_solve(L, B, w.tile, fixed=fixed)
    check(w, X, L, B)


def test_default_tile_in_place_and_repeatable():
    w = TW("p", 900, 130, 256, seed=31)
    L, B = inputs.make_trsm_operands(w)
    X0 = gpu_solve(L, B, 0)
    check(w, X0, L, B)
    assert (gpu_solve(L, B, 256) == X0).all()              # tile 0 selects 256
    assert (gpu_solve(L, B, 0, in_place=True) == X0).all()
    assert (gpu_solve(L, B, 0) == X0).all()                # run to run identical


def test_exact_cases():
    import torch
    from paper_2511_09987_b200 import binding
    # unit lower-triangular integer L and integer X: every fp32 intermediate is exact on the chain path
    r = np.random.default_rng(5)
    n, m = 300, 17
    L = np.tril(r.integers(-1, 2, size=(n, n))).astype(np.float32)
    L[np.arange(n), np.arange(n)] = 1.0
    L[np.triu_indices(n, 1)] = np.nan
    keep = np.tril(r.random((n, n)) < 8.0 / n, -1)            # sparse coupling keeps the integers small
    L = np.where(np.tril(np.ones((n, n), dtype=bool), -1) & ~keep, np.float32(0), L)
    Xt = r.integers(-2, 3, size=(n, m)).astype(np.float64)
    Bm = np.tril(np.nan_to_num(L)).astype(np.float64) @ Xt
    assert np.abs(Bm).max() < 2 ** 20
    for tile in (32, 100, 256):
        for fixed in (True, False):
            X = gpu_solve(L, Bm.astype(np.float32), tile, fixed=fixed)
            assert (X == Xt.astype(np.float32)).all(), (tile, fixed)
    # identity and diagonal
    Bd = r.standard_normal((n, m)).astype(np.float32)
    assert (gpu_solve(np.eye(n, dtype=np.float32), Bd, 64) == Bd).all()
    del torch, binding


def test_full_size_every_column():
    """t2 at full size: the forward comparison with the oracle on all 4096 right-hand-side columns (every output of
    X), the fp64 residual on one column of every 32-column CTA of the diagonal-tile kernel."""
    import os
    w = inputs.TRSM_WORKLOADS["t2"]
    L, B = inputs.make_trsm_operands(w)
    X = gpu_solve(L, B, w.tile)
    assert X.shape == B.shape and np.isfinite(X).all()
    threads = os.cpu_count() or 8
    rcols = np.arange(0, w.m, 32) + (np.arange(w.m // 32) * 7) % 32      # one column per CTA, at varying offsets
    R, S = otrsm.residual(L, B, X, rcols)
    assert (np.abs(R) <= 1e-5 * S).all(), "residual %g of its scale" % float((np.abs(R) / S).max())
    absL = np.abs(np.tril(np.nan_to_num(L))).astype(np.float64)
    assert w.coupling == "dominant"
    for c0 in range(0, w.m, 512):
        cols = np.arange(c0, min(w.m, c0 + 512))
        ref = otrsm.block_trsm(L, np.ascontiguousarray(B[:, cols]), w.tile, threads=threads)
        err = np.abs(X[:, cols].astype(np.float64) - ref)
        # the residual scale |B| + |L||X| of these columns (a library product: it is only the yardstick); with
        # |L^-1| <= 2 in the infinity norm a column's error is at most twice its largest admissible residual
        Sc = np.abs(B[:, cols]).astype(np.float64) + absL @ np.abs(X[:, cols]).astype(np.float64)
        bound = 2e-5 * Sc.max(axis=0, keepdims=True)
        assert (err <= bound).all(), "forward error %g of its bound (columns %d..)" % (float((err / bound).max()), c0)


def test_quick_full_size_sampled_columns():
    w = inputs.TRSM_WORKLOADS["t2"]
    L, B = inputs.make_trsm_operands(w)
    X = gpu_solve(L, B, w.tile)
    cols = [0, 1, 31, 32, 255, 256, 1000, 2047, 2048, 3071, 4064, 4095]
    check(w, X, L, B, cols=cols, threads=12)
