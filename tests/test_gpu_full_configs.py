"""The five workload configurations at full size, in the launch configuration the
benchmark times, compared with the oracle on EVERY output: the whole of C is walked
by the collapsed oracle in blocks of rows (int8 bit for bit; fp32 under the
fixed-k-order flag bit for bit against the fused chain, else within 1e-5 S; bf16
within 4e-3 S, S_ij = sum_k |A_ik||B_kj|).  The `quick` variants check sampled rows
only and exist for fast iteration on a kernel."""
import os

import numpy as np
import pytest

import oracle
from paper_2511_09987_b200 import inputs
from parity_util import TOL, check_workload, compare_rows, gpu_run

pytestmark = pytest.mark.gpu
W = inputs.WORKLOADS
THREADS = os.cpu_count() or 8


def check_every_output(w, fixed_k_order=None, block_rows=1024):
    """All M x N outputs of every problem of `w` against the oracle, `block_rows` rows of C at a time."""
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B, fixed_k_order)
    fixed = w.fixed_k_order if fixed_k_order is None else fixed_k_order
    exact = w.dtype == "f32" and fixed
    worst, checked = 0.0, 0
    for b in (range(w.batch) if w.batch > 1 else [None]):
        Ab, Bb, Cb = (A, B, C) if b is None else (A[b], B[b], C[b])
        assert Cb.shape == (w.M, w.N)
        for r0 in range(0, w.M, block_rows):
            rows = np.arange(r0, min(w.M, r0 + block_rows))
            worst = max(worst, compare_rows(w, Ab, Bb, Cb[rows], rows, THREADS, exact))
            checked += rows.size * w.N
    assert checked == w.batch * w.M * w.N
    return worst


def test_c1_fp32_64_every_output_bit_exact():
    check_every_output(W["c1"])


def test_c2_int8_4096_every_output_bit_exact():
    check_every_output(W["c2"])


def test_c3_bf16_8192_every_output():
    assert check_every_output(W["c3"], block_rows=512) < TOL["bf16"]


def test_c4_fp32_tall_skinny_every_output_strict_and_default():
    check_every_output(W["c4"], fixed_k_order=True, block_rows=8192)    # bit-equal to the fused chain
    assert check_every_output(W["c4"], fixed_k_order=False, block_rows=8192) < TOL["f32"]


def test_c5_batched_bf16_every_problem():
    w = W["c5"]
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B)
    assert C.shape == (1024, 256, 256)
    for b in range(w.batch):
        ref = oracle.collapsed("bf16", A[b], B[b], threads=THREADS)
        S, _ = oracle.abs_sum_rows("bf16", A[b], B[b], threads=THREADS)
        assert (np.abs(C[b].astype(np.float64) - ref) <= TOL["bf16"] * S).all(), b


# ---- quick variants: sampled rows (always including tile edges), for iterating on one kernel
def test_quick_c2_sampled_rows():
    check_workload(W["c2"], rows_per_problem=48)


def test_quick_c3_sampled_rows():
    assert check_workload(W["c3"], rows_per_problem=20) < TOL["bf16"]


def test_quick_c4_sampled_rows():
    check_workload(W["c4"], rows_per_problem=2048, fixed_k_order=True)
    check_workload(W["c4"], rows_per_problem=2048, fixed_k_order=False)
