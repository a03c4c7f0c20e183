"""Prefix-sum recurrence on the GPU against the CPU oracle on the same seeded inputs.

int32: bit-exact (wrap-around arithmetic is associative, so any grouping gives the same bits).
float32: ``|P_i - P_oracle_i| <= 1e-6 * S_i`` with ``S_i = sum_{k<=i} |A_k|`` and the oracle's walk in fp64.  Derivation:
the GPU forms fp32 sums only inside the 128 consecutive elements a warp owns: 3 additions inside a group of four, 5 across
the lanes, 1 to combine them, each with relative error 2^-24 on a partial sum bounded by the ``|A|`` mass it covers; sums
of 128 elements, tile sums and the value carried from tile to tile are fp64 (descriptors keep 50 significand bits); the
final ``head + (tail + y)`` adds one rounding relative to the warp's own mass and one relative to ``|P_i|``.  Together at
most ``11 * 2^-24 * S_i = 6.6e-7 * S_i``, whatever the length of the sequence.
"""
import numpy as np
import pytest

from oracle import scan as oscan
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu
SW = inputs.ScanWorkload
TOL = 1e-6


def gpu_scan(A, *, in_place=False, pitch=None):
    import torch
    from paper_2511_09987_b200 import binding
    if pitch is None:
        dA = torch.from_numpy(np.ascontiguousarray(A)).cuda()
    else:  # rows with a pitch larger than n, poisoned padding
        rows, n = A.shape
        buf = torch.full((rows, pitch), 7, dtype=torch.from_numpy(A[:0]).dtype, device="cuda")
        buf[:, :n] = torch.from_numpy(A).cuda()
        dA = buf[:, :n]
    P = binding.prefix_sum(dA, dA if in_place else None)
    assert binding.last_device_status() == binding.CYC_OK
    torch.cuda.synchronize()
    if pitch is not None and in_place:
        assert (buf[:, A.shape[1]:] == 7).all(), "the padding between rows was written"
    return P.cpu().numpy()


def check(P, A):
    if A.dtype == np.int32:
        ref = oscan.prefix_sum(A, arithmetic="i32")
        assert P.dtype == np.int32 and P.tobytes() == ref.tobytes()
        return 0.0
    ref, S = oscan.prefix_sum(A, arithmetic="f64", with_scale=True)
    assert P.dtype == np.float32 and np.isfinite(P).all()
    err = np.abs(P.astype(np.float64) - ref)
    assert (err <= TOL * S).all(), "max error %g of S (tolerance %g)" % (float((err / np.maximum(S, 1e-300)).max()), TOL)
    return float((err / np.maximum(S, 1e-300)).max())


CASES = [SW("one", 1, 1, "f32", 60), SW("one_i", 1, 1, "i32", 61), SW("three", 1, 3, "f32", 62), SW("quarter_minus_1", 1, 4095, "i32", 63),
         SW("quarter", 1, 4096, "f32", 64), SW("quarter_plus_1", 1, 4097, "f32", 65), SW("ragged", 1, 10001, "i32", 66),
         SW("tile_minus_1", 1, 16383, "f32", 74), SW("tile", 2, 16384, "i32", 75), SW("tile_plus_1", 1, 16385, "f32", 76),
         SW("tile_plus_quarter", 3, 16384 + 4096, "f32", 77),
         SW("p1", 3, 10000, "f32", 30), SW("odd_rows", 7, 4099, "i32", 67), SW("short_rows", 500, 37, "f32", 68),
         SW("many_tiles", 1, 40 * 16384 + 13, "f32", 69), SW("many_tiles_i", 2, 70 * 16384 + 4097, "i32", 70),
         SW("long_lookback", 1, 3000 * 4096 + 5, "f32", 71),
         # long rows: hundreds of tiles per row, several rows
         SW("long_row_exact", 1, 1 << 22, "i32", 78), SW("long_rows_ragged", 3, (1 << 22) + 12345, "f32", 79),
         SW("long_row_two_sections", 1, 6_000_000 + 3, "i32", 94), SW("long_row_three_sections", 2, 11_000_000 + 1, "f32", 95)]


@pytest.mark.parametrize("w", CASES, ids=[c.name for c in CASES])
def test_against_the_oracle(w):
    A = inputs.make_scan_operand(w)
    check(gpu_scan(A), A)


@pytest.mark.parametrize("dtype", ["f32", "i32"])
def test_in_place_unaligned_and_pitched(dtype):
    A = inputs.make_scan_operand(SW("x", 5, 9001, dtype, 72))
    check(gpu_scan(A, in_place=True), A)
    check(gpu_scan(A, pitch=9003), A)                    # rows not 16-byte aligned: the scalar path
    check(gpu_scan(A, pitch=9008, in_place=True), A)     # aligned rows, padding untouched
    import torch
    from paper_2511_09987_b200 import binding
    flat = torch.from_numpy(A.reshape(-1)).cuda()
    P = binding.prefix_sum(flat[1:])                     # base pointer off the 16-byte grid
    check(P.cpu().numpy()[None, :], A.reshape(1, -1)[:, 1:])


def test_long_rows_in_place_and_pitched():
    A = inputs.make_scan_operand(SW("x", 2, (1 << 22) + 77, "f32", 96))
    check(gpu_scan(A, in_place=True), A)
    check(gpu_scan(A, pitch=(1 << 22) + 79), A)          # rows not 16-byte aligned: the scalar path


def test_closed_forms_and_exact_cases():
    n = 3 * 16384 + 77
    ones = np.ones((2, n), dtype=np.float32)
    assert (gpu_scan(ones) == np.arange(1, n + 1, dtype=np.float32)).all()          # exact: every partial sum is an integer < 2^24
    assert (gpu_scan(ones.astype(np.int32)) == np.arange(1, n + 1)).all()
    alt = np.where(np.arange(n) % 2 == 0, 1, -1).astype(np.float32)[None, :]
    assert (gpu_scan(alt) == ((np.arange(n) + 1) % 2)).all()
    # the carried value exceeds fp32's integer range: 2^24 ones followed by ones still count exactly up to rounding of P_i
    big = np.ones((1, (1 << 24) + 4096), dtype=np.float32)
    P = gpu_scan(big)
    want = np.arange(1, big.shape[1] + 1, dtype=np.float64)
    assert (P == want.astype(np.float32)).all()         # each P_i is the exact integer rounded once to fp32
    # wrap-around
    w = np.full((1, 5000), 2 ** 31 - 1, dtype=np.int32)
    assert gpu_scan(w).tobytes() == oscan.prefix_sum(w, arithmetic="i32").tobytes()
    # int32 is run-to-run identical
    A = inputs.make_scan_operand(SW("r", 3, 100000, "i32", 73))
    assert gpu_scan(A).tobytes() == gpu_scan(A).tobytes()


def test_arguments():
    import torch
    from paper_2511_09987_b200 import binding as b
    x = torch.zeros(100, dtype=torch.float32, device="cuda")
    y = torch.zeros(100, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert b.cyc_prefix_sum(1, 0, b.CYC_F32, x.data_ptr(), 0, y.data_ptr(), 0, s, 0) == b.CYC_ERR_INVALID_ARG
    assert b.cyc_prefix_sum(1, 100, b.CYC_F32, x.data_ptr(), 0, None, 0, s, 0) == b.CYC_ERR_INVALID_ARG
    assert b.cyc_prefix_sum(1, 100, b.CYC_F32, x.data_ptr(), 0, y.data_ptr(), 0, s, 1) == b.CYC_ERR_INVALID_ARG
    assert b.cyc_prefix_sum(2, 50, b.CYC_F32, x.data_ptr(), 40, y.data_ptr(), 0, s, 0) == b.CYC_ERR_INVALID_ARG       # stride < n
    assert b.cyc_prefix_sum(1, 60, b.CYC_F32, x.data_ptr(), 0, x.data_ptr() + 40, 0, s, 0) == b.CYC_ERR_INVALID_ARG    # partial overlap
    assert b.cyc_prefix_sum(1, 100, b.CYC_BF16_F32, x.data_ptr(), 0, y.data_ptr(), 0, s, 0) == b.CYC_ERR_UNSUPPORTED
    assert b.cyc_prefix_sum(1, 100, 9, x.data_ptr(), 0, y.data_ptr(), 0, s, 0) == b.CYC_ERR_INVALID_ARG


def test_full_size_workloads():
    """p2 (one sequence of 2^28 floats) element by element against the fp64 walk; p3 (4096 x 65536 int32) bit for bit."""
    w = inputs.SCAN_WORKLOADS["p2"]
    A = inputs.make_scan_operand(w)
    worst = check(gpu_scan(A), A)
    assert worst < TOL
    w = inputs.SCAN_WORKLOADS["p3"]
    A = inputs.make_scan_operand(w)
    check(gpu_scan(A), A)
