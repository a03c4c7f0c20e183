"""The schedules of the matrix-multiply recurrence on the GPU against the oracle's walkers of the same schedules.

Section "Space-time Mappings of Dataflow Recurrences" prints two programs for the one base recurrence: the
weight-stationary one (cells (i,k), time j) and the output-stationary one (cells (i,j) keep C_ij, k runs in time).
Every kernel of the library keeps its block of C in place for the whole k loop (in tensor memory or registers) and
streams A and B past it: as a space-time mapping that IS the output-stationary program, with a CTA tile as the block of
cells.  This file pins that reading: the kernels must reproduce the oracle's `os_cannon` walker -- bit for bit where the
arithmetic allows it (int8 on the tensor cores; fp32 under the fixed-k-order flag against the fused chain) and within the
stated tolerance for bf16 -- on ragged shapes that span several tiles, exactly as they reproduce the weight-stationary
walker.  The k-sliced schedule (partial sums of different k ranges held by different cells and combined in k order) is
checked against the same walker.
"""
import numpy as np
import pytest

import oracle
from paper_2511_09987_b200 import inputs
from parity_util import TOL, gpu_run

pytestmark = pytest.mark.gpu


def _w(dtype, M, N, K, seed, col=False, fixed=False):
    if dtype == "i8":
        return inputs.Workload("sched", "i8", M, N, K, seed, 1, col, fixed, ("int8",), ("int8",))
    return inputs.Workload("sched", dtype, M, N, K, seed, 1, col, fixed, ("uniform", -1.0, 1.0), ("normal", 1.0))


INT8_CASES = [(130, 136, 160, True), (100, 272, 144, False), (260, 264, 272, True), (300, 528, 400, False), (515, 260, 144, True)]


@pytest.mark.parametrize("M,N,K,col", INT8_CASES)
def test_int8_tensor_core_kernels_equal_the_output_stationary_walker(M, N, K, col):
    from paper_2511_09987_b200 import binding
    w = _w("i8", M, N, K, seed=60 + M, col=col)
    A, B = inputs.make_operands(w)
    assert binding.kernel_for(1, M, N, K, "i8", b_col_major=col).startswith("tcgen05")
    assert binding.schedule_for(1, M, N, K, "i8", b_col_major=col) == "output_stationary"
    C = gpu_run(w, A, B)
    os_c = oracle.walk("os_cannon", "i8", A, B, b_col_major=col)
    ws_c = oracle.walk("literal", "i8", A, B, b_col_major=col) if M * N * K < 3e6 else oracle.collapsed("i8", A, B, b_col_major=col)
    assert C.tobytes() == os_c.tobytes()
    assert C.tobytes() == ws_c.tobytes()


@pytest.mark.parametrize("M,N,K", [(64, 64, 64), (130, 70, 90), (257, 129, 65), (300, 520, 77)])
def test_strict_fp32_kernel_equals_the_output_stationary_walker_bit_for_bit(M, N, K):
    from paper_2511_09987_b200 import binding
    w = _w("f32", M, N, K, seed=70 + M, fixed=True)
    A, B = inputs.make_operands(w)
    assert binding.kernel_for(1, M, N, K, "f32", fixed_k_order=True) == "simt"
    assert binding.schedule_for(1, M, N, K, "f32", fixed_k_order=True) == "output_stationary"
    C = gpu_run(w, A, B)
    assert C.tobytes() == oracle.walk("os_cannon", "f32", A, B, fma=True).tobytes()
    # and within the stated tolerance of the two-rounding reading of the same program
    ref = oracle.walk("os_cannon", "f32", A, B, fma=False)
    S, _ = oracle.abs_sum_rows("f32", A, B)
    assert (np.abs(C.astype(np.float64) - ref) <= TOL["f32"] * S).all()


@pytest.mark.parametrize("M,N,K", [(130, 136, 160), (260, 264, 272), (515, 264, 136)])
def test_bf16_tensor_core_kernels_against_the_output_stationary_walker(M, N, K):
    from paper_2511_09987_b200 import binding
    w = _w("bf16", M, N, K, seed=80 + M)
    A, B = inputs.make_operands(w)
    assert binding.kernel_for(1, M, N, K, "bf16").startswith("tcgen05")
    C = gpu_run(w, A, B)
    ref = oracle.walk("os_cannon", "bf16", A, B)
    S, _ = oracle.abs_sum_rows("bf16", A, B)
    assert (np.abs(C.astype(np.float64) - ref) <= TOL["bf16"] * S).all()


def test_k_sliced_schedule_equals_the_walkers_for_int8():
    """Split-K: the k range of a tile is cut into slices held by different CTA pairs and the partial sums are added in
    increasing k.  Integer addition is associative, so the result must still be the walkers' bit for bit."""
    from paper_2511_09987_b200 import binding
    M, N, K = 260, 300, 4224      # four tiles, 33 k-blocks of 128
    w = _w("i8", M, N, K, seed=90, col=True)
    A, B = inputs.make_operands(w)
    assert binding.kernel_for(1, M, N, K, "i8", b_col_major=True) == "tcgen05_pair_splitk"
    assert binding.schedule_for(1, M, N, K, "i8", b_col_major=True) == "k_sliced"
    assert binding.schedule_for(1, M, N, K, "i8", b_col_major=True, fixed_k_order=True) == "output_stationary"
    C = gpu_run(w, A, B)
    assert C.tobytes() == oracle.collapsed("i8", A, B, b_col_major=True, threads=8).tobytes()
    rows = np.array([0, 127, 128, 259])
    os_rows = oracle.walk("os_cannon", "i8", A[rows], B, b_col_major=True)
    assert (C[rows] == os_rows).all()


TAIL_CASES = [
    # dtype, batch, M, N, K, col   -- tile counts that leave a remainder of at most half the 74 CTA pairs
    ("i8", 1, 2500, 2600, 2048, True),      # 10 x 11 = 110 tiles, remainder 36: two slices of 8 k-blocks
    ("bf16", 1, 2500, 2344, 1032, False),   # 100 tiles, remainder 26; 17 k-blocks: slices of 9 and 8
    ("i8", 3, 1280, 1536, 4096, False),     # 3 x 30 tiles, remainder 16: four slices of 8 k-blocks
    ("bf16", 1, 2304, 2560, 1096, True),    # 90 tiles, remainder 16; 18 k-blocks, the last ragged: slices of 9
]


@pytest.mark.parametrize("dtype,batch,M,N,K,col", TAIL_CASES)
def test_sliced_tail_every_output(dtype, batch, M, N, K, col):
    """The leftover tiles of the last round are cut into k-slices spread over all CTA pairs and summed in increasing
    k by whichever pair finishes a strip last: int8 must equal the walkers bit for bit, bf16 stay within tolerance, and
    the result must not depend on which pair was last (two launches, two streams, identical bits)."""
    import torch
    from paper_2511_09987_b200 import binding
    dist = ("int8",) if dtype == "i8" else ("uniform", -1.0, 1.0)
    w = inputs.Workload("tail", dtype, M, N, K, 95 + batch, batch, col, False, dist, dist)
    assert binding.kernel_for(batch, M, N, K, dtype, b_col_major=col) == "tcgen05_pair"
    assert binding.schedule_for(batch, M, N, K, dtype, b_col_major=col) == "output_stationary+k_sliced_tail"
    assert binding.schedule_for(batch, M, N, K, dtype, b_col_major=col, fixed_k_order=True) == "output_stationary"
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B)
    C2 = gpu_run(w, A, B)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        C3 = gpu_run(w, A, B)
    assert C.tobytes() == C2.tobytes() == C3.tobytes()
    C1 = gpu_run(w, A, B, fixed_k_order=True)          # one owner per output: the plain schedule
    for b in range(batch):
        Ab, Bb, Cb, C1b = (A, B, C, C1) if batch == 1 else (A[b], B[b], C[b], C1[b])
        ref = oracle.collapsed(dtype, Ab, Bb, b_col_major=col, threads=16)
        if dtype == "i8":
            assert Cb.tobytes() == ref.tobytes()
            assert C1b.tobytes() == ref.tobytes()
        else:
            S, _ = oracle.abs_sum_rows(dtype, Ab, Bb, b_col_major=col, threads=16)
            assert (np.abs(Cb.astype(np.float64) - ref) <= TOL[dtype] * S).all()
            assert (np.abs(C1b.astype(np.float64) - ref) <= TOL[dtype] * S).all()


def test_headline_int8_configuration_uses_the_sliced_tail():
    from paper_2511_09987_b200 import binding
    assert binding.schedule_for(1, 4096, 4096, 4096, "i8", b_col_major=True) == "output_stationary+k_sliced_tail"
    assert binding.schedule_for(1024, 256, 256, 256, "bf16") == "output_stationary"     # remainder 62 of 74: no slicing
    assert binding.schedule_for(1, 8192, 8192, 8192, "bf16") == "output_stationary"     # tall tiles


def test_caller_supplied_result_is_checked_before_it_reaches_a_kernel():
    import torch
    from paper_2511_09987_b200 import binding
    A = torch.zeros((64, 32), dtype=torch.float32, device="cuda")
    B = torch.zeros((32, 48), dtype=torch.float32, device="cuda")
    for bad in (torch.empty((64, 47), dtype=torch.float32, device="cuda"), torch.empty((64, 48), dtype=torch.int32, device="cuda"),
                torch.empty((64, 48), dtype=torch.float32), torch.empty((48, 64), dtype=torch.float32, device="cuda").t()):
        with pytest.raises(ValueError):
            binding.recurrence_matmul(A, B, bad)
    Q = torch.zeros((2, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):
        binding.flash_attention(Q, Q, Q, torch.empty((2, 128, 63), dtype=torch.float32, device="cuda"))
