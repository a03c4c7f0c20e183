"""Seeded random shapes, strides, offsets and options for the recurrences beyond the matrix product: each case is checked
against its oracle with the tolerance of the kernel's own test file.  Meant to catch what the hand-picked cases miss
(odd pitches, unaligned bases, ragged tiles in combination with in-place operation or the fixed-order flag)."""
import numpy as np
import pytest

from oracle import chol as ochol
from oracle import fa2 as ofa2
from oracle import scan as oscan
from oracle import trsm as otrsm
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu


def test_prefix_sum_random_cases():
    import torch
    from paper_2511_09987_b200 import binding
    rng = np.random.default_rng(2024)
    for it in range(40):
        rows = int(rng.choice([1, 2, 3, 7, 33, 200]))
        n = int(rng.choice([1, 5, 4095, 4096, 4097, 8191, 8193, 16384, 16385, 40000, 262144, 262145, 300001, 1000003]))
        if rows * n > 2e7:
            rows = max(1, int(2e7 // n))
        dt = str(rng.choice(["f32", "i32"]))
        pitch = n + int(rng.choice([0, 0, 1, 3, 4, 8]))
        off = int(rng.choice([0, 0, 1, 4]))
        in_place = bool(rng.integers(0, 2))
        A = inputs.make_scan_operand(inputs.ScanWorkload("z", rows, n, dt, 1000 + it))
        buf = torch.zeros(off + rows * pitch, dtype=torch.from_numpy(A).dtype, device="cuda")
        view = buf[off:].view(rows, pitch)[:, :n]
        view.copy_(torch.from_numpy(A).cuda())
        P = binding.prefix_sum(view, view if in_place else None).cpu().numpy()
        assert binding.last_device_status() == binding.CYC_OK
        what = (rows, n, dt, pitch, off, in_place)
        if dt == "i32":
            assert P.tobytes() == oscan.prefix_sum(A, arithmetic="i32").tobytes(), what
        else:
            ref, S = oscan.prefix_sum(A, arithmetic="f64", with_scale=True)
            assert (np.abs(P - ref) <= 1e-6 * S).all(), what


def test_cholesky_random_cases():
    import torch
    from paper_2511_09987_b200 import binding
    rng = np.random.default_rng(2025)
    for it in range(24):
        n = int(rng.choice([1, 2, 31, 32, 33, 64, 100, 255, 256, 257, 300, 511, 512, 513, 777, 1024, 1500]))
        tile = int(rng.choice([0, 0, 256, 128, 64, 32, 17, 5])) if n <= 600 else int(rng.choice([0, 256, 128, 100]))
        coupling = str(rng.choice(["wigner", "dominant"]))
        in_place, fixed = bool(rng.integers(0, 2)), bool(rng.integers(0, 4) == 0)
        A = inputs.make_chol_operand(inputs.CholWorkload("z", n, tile, 2000 + it, coupling))
        dA = torch.from_numpy(A).cuda()
        L = binding.cholesky(dA, dA if in_place else None, tile=tile, fixed_k_order=fixed).cpu().numpy()
        assert binding.last_device_status() == binding.CYC_OK
        what = (n, tile, coupling, in_place, fixed)
        R, S = ochol.residual(A, L, np.arange(n))
        assert np.isfinite(L[np.tril(np.ones((n, n), bool))]).all(), what
        assert (np.abs(R) <= 1e-5 * S + 1e-30).all(), what
        if not in_place:
            assert (np.triu(L, 1) == 0).all(), what


def test_attention_random_cases():
    import torch
    from paper_2511_09987_b200 import binding
    rng = np.random.default_rng(2026)
    for it in range(24):
        d, batch = int(rng.choice([64, 128])), int(rng.choice([1, 2, 5]))
        N = int(rng.choice([1, 2, 127, 128, 129, 255, 300, 513]))
        M = int(rng.choice([1, 2, 63, 64, 65, 127, 128, 129, 255, 256, 257, 700, 1025]))
        w = inputs.AttentionWorkload("z", batch, N, M, d, seed=3000 + it, qk_std=float(rng.choice([0.05, 1.0, 3.0])))
        Q, K, V = inputs.make_attention_operands(w)
        O = binding.flash_attention(*(torch.from_numpy(x).view(torch.bfloat16).cuda() for x in (Q, K, V))).cpu().numpy()
        assert binding.last_device_status() == binding.CYC_OK
        for b in range(batch):
            ref, _, _, scale = ofa2.attention(Q[b], K[b], V[b], 128, threads=8, with_state=True)
            assert (np.abs(O[b] - ref) <= 4e-3 * scale + 1e-30).all(), (batch, N, M, d, w.qk_std)


def test_triangular_solve_random_cases():
    import torch
    from paper_2511_09987_b200 import binding
    rng = np.random.default_rng(2027)
    for it in range(16):
        n = int(rng.choice([1, 33, 255, 256, 257, 500, 1000]))
        m = int(rng.choice([1, 31, 32, 33, 100, 257]))
        tile = int(rng.choice([0, 256, 64, 37]))
        w = inputs.TrsmWorkload("z", n, m, tile or 256, seed=4000 + it, coupling=str(rng.choice(["dominant", "sqrt"])))
        L, B = inputs.make_trsm_operands(w)
        X = binding.block_trsm(torch.from_numpy(L).cuda(), torch.from_numpy(B).cuda(), tile=tile).cpu().numpy()
        assert binding.last_device_status() == binding.CYC_OK
        R, S = otrsm.residual(L, B, X, np.arange(m))
        assert (np.abs(R) <= 1e-5 * S + 1e-30).all(), (n, m, tile, w.coupling)
