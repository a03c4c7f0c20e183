"""Tiled Cholesky recurrence on the GPU against the fp64 oracle on the same seeded inputs.

Tolerances.  Backward: ``|A - L L^T|_ij <= 1e-5 (|L||L|^T)_ij`` element by element on the lower triangle -- the
factorisation in fp32 is backward stable with ``|dA| <= gamma_(n+1) |L||L|^T`` (worst case ``(n+1) 2^-24``, about
``sqrt(n) 2^-24 = 5e-6`` for random data at n = 8192), and the tensor-core path of the SYRK / GEMM sums stays below
``2e-6`` of the same scale; 1e-5 is the fp32 tolerance of the multiply path.  Forward: ``|L - L_oracle|_ij <= 1e-4
sqrt(A_ii)``: the relative change of the factor is bounded by about ``kappa(A) / sqrt(2)`` times the relative backward
error, the input recipes have ``kappa(A) <= 6``, and ``sqrt(A_ii)`` is the norm of row i of L.  Exact cases (integer
factors) must be reproduced exactly.
"""
from math import comb

import numpy as np
import pytest

from oracle import chol as ochol
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu
CW = inputs.CholWorkload


def gpu_chol(A, tile=0, *, in_place=False, fixed_k_order=False):
    import torch
    from paper_2511_09987_b200 import binding
    dA = torch.from_numpy(np.ascontiguousarray(A)).cuda()
    L = binding.cholesky(dA, dA if in_place else None, tile=tile, fixed_k_order=fixed_k_order)
    assert binding.last_device_status() == binding.CYC_OK
    torch.cuda.synchronize()
    return L.cpu().numpy()


def check(L, A, tile, rows=None, threads=8, ref=None):
    n = A.shape[0]
    rows = np.arange(n) if rows is None else np.asarray(rows)
    low = np.tril(np.ones((n, n), dtype=bool))
    assert np.isfinite(L[low]).all()
    R, S = ochol.residual(A, L, rows)
    assert (np.abs(R) <= 1e-5 * S + 1e-30).all(), "backward: max %g of |L||L|^T" % float((np.abs(R) / np.maximum(S, 1e-300)).max())
    if ref is None:
        ref = ochol.cholesky(A, tile or 256, threads=threads)
    scale = np.sqrt(np.diag(A).astype(np.float64))[rows, None]
    err = np.where(low[rows], np.abs(L[rows].astype(np.float64) - ref[rows]), 0.0)   # above the diagonal is not compared
    assert (err <= 1e-4 * scale).all(), "forward: max %g of sqrt(A_ii)" % float((err / scale).max())
    return float((np.abs(R) / np.maximum(S, 1e-300)).max()), float((err / scale).max())


CASES = [CW("one", 1, 0, 80), CW("two", 2, 0, 81), CW("sub_block", 33, 0, 82), CW("one_tile", 256, 0, 83), CW("tile_plus_1", 257, 0, 84),
         CW("h1", 600, 64, 50), CW("dominant", 700, 128, 85, "dominant"), CW("ragged_256", 1000, 0, 86), CW("tile_7", 100, 7, 87),
         CW("unaligned_n", 1027, 0, 88), CW("wide", 2048, 0, 89)]


@pytest.mark.parametrize("w", CASES, ids=[c.name for c in CASES])
def test_against_the_oracle(w):
    A = inputs.make_chol_operand(w)
    L = gpu_chol(A, w.tile)
    assert (np.triu(L, 1) == 0).all(), "entries above the diagonal must be zero"
    check(L, A, w.tile)


def test_in_place_and_fixed_order():
    w = CW("p", 900, 128, 90)
    A = inputs.make_chol_operand(w)
    L = gpu_chol(A, w.tile, in_place=True)
    up = np.triu_indices(w.n, 1)
    assert np.isnan(L[up]).all(), "in place: entries above the diagonal stay as they were"
    check(L, A, w.tile)
    a = gpu_chol(A, w.tile, fixed_k_order=True)
    b = gpu_chol(A, w.tile, fixed_k_order=True)
    assert a.tobytes() == b.tobytes()
    check(a, A, w.tile)


def test_closed_forms_and_exact_cases():
    n = 300
    i = np.arange(n)
    A = (np.minimum.outer(i, i) + 1).astype(np.float32)          # factor: the all-ones lower triangle
    for tile in (0, 64):
        assert (gpu_chol(A, tile) == np.tril(np.ones((n, n), dtype=np.float32))).all()
    P = np.array([[comb(a + b, a) for b in range(11)] for a in range(11)], dtype=np.float32)
    want = np.array([[comb(a, b) if b <= a else 0 for b in range(11)] for a in range(11)], dtype=np.float32)
    assert (gpu_chol(P) == want).all()
    r = np.random.default_rng(4)
    L0 = np.tril(r.integers(-3, 4, size=(400, 400))).astype(np.int64)
    L0[np.arange(400), np.arange(400)] = 2 ** r.integers(0, 3, size=400)   # powers of two: the reciprocal scaling of the
    Ai = (L0 @ L0.T).astype(np.float32)                                     # tiles below the diagonal is then exact too
    assert (gpu_chol(Ai, 128) == L0).all()
    rho = 0.5
    A = (rho ** np.abs(np.subtract.outer(i, i))).astype(np.float32)
    want = np.tril(rho ** np.subtract.outer(i, i).clip(0).astype(np.float64)) * np.sqrt(1 - rho * rho)
    want[:, 0] = rho ** i
    assert np.abs(gpu_chol(A, 64) - want).max() <= 1e-6
    # not positive definite: NaN from the square root of a negative pivot, no error and no hang
    bad = gpu_chol(np.array([[1.0, 2.0], [2.0, 1.0]], dtype=np.float32))
    assert bad[0, 0] == 1.0 and bad[1, 0] == 2.0 and np.isnan(bad[1, 1])


def test_full_size_sampled_rows():
    w = inputs.CHOL_WORKLOADS["h2"]
    A = inputs.make_chol_operand(w)
    L = gpu_chol(A, w.tile)
    rows = np.array([0, 1, 255, 256, 257, 1000, 4095, 4096, 6000, 8190, 8191])
    ref = ochol.cholesky(A, w.tile, threads=16)
    back, fwd = check(L, A, w.tile, rows=rows, ref=ref)
    assert back < 1e-5 and fwd < 1e-4
