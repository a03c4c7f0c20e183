"""The five workload configurations at full size, in the launch configuration the
benchmark times, checked on sampled rows of C that the oracle computes one by one
(every sampled row covers all n-tiles; the sample always includes tile edges)."""
import pytest

from paper_2511_09987_b200 import inputs
from parity_util import check_workload

pytestmark = pytest.mark.gpu
W = inputs.WORKLOADS


def test_c2_int8_4096_bit_exact():
    check_workload(W["c2"], rows_per_problem=48)


def test_c3_bf16_8192():
    worst = check_workload(W["c3"], rows_per_problem=20)
    assert worst < 4e-3


def test_c4_fp32_tall_skinny_strict_and_default():
    check_workload(W["c4"], rows_per_problem=2048, fixed_k_order=True)   # bit-exact chain
    check_workload(W["c4"], rows_per_problem=2048, fixed_k_order=False)


def test_c5_batched_bf16():
    import numpy as np
    import oracle
    from parity_util import gpu_run, TOL
    w = W["c5"]
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B)
    assert C.shape == (1024, 256, 256)
    for b in list(range(0, 1024, 37)) + [1023]:          # 29 whole problems, first and last included
        ref = oracle.collapsed("bf16", A[b], B[b], threads=8)
        S, _ = oracle.abs_sum_rows("bf16", A[b], B[b], threads=8)
        assert (np.abs(C[b].astype(np.float64) - ref) <= TOL["bf16"] * S).all(), b
