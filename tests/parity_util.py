"""Shared helpers of the GPU parity tests: run a workload through the C ABI and
compare with the CPU oracle on the same seeded operands."""
import numpy as np

import oracle
from paper_2511_09987_b200 import inputs

# tolerances of the acceptance criterion, as multiples of S_ij = sum_k |A_ik||B_kj|
TOL = {"f32": 1e-5, "bf16": 4e-3}
NP_IN = {"f32": np.float32, "bf16": np.uint16, "i8": np.int8}


def to_device(x, dtype):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype == "bf16":
        t = t.view(torch.bfloat16)
    return t.cuda()


def gpu_run(w, A, B, fixed_k_order=None):
    """Evaluate workload ``w`` on the GPU through the binding; returns a host numpy array."""
    import torch
    from paper_2511_09987_b200 import binding
    fixed = w.fixed_k_order if fixed_k_order is None else fixed_k_order
    dA, dB = to_device(A, w.dtype), to_device(B, w.dtype)
    if w.batch > 1:
        C = binding.recurrence_matmul_batched(dA, dB, b_col_major=w.b_col_major, fixed_k_order=fixed)
    else:
        C = binding.recurrence_matmul(dA, dB, b_col_major=w.b_col_major, fixed_k_order=fixed)
    assert binding.last_device_status() == binding.CYC_OK
    torch.cuda.synchronize()
    return C.cpu().numpy()


def compare_rows(w, A, B, C_gpu_rows, rows, threads=8, expect_bit_exact_fma=False):
    """Compare rows of one (un-batched) problem with the oracle.  Returns the largest normalised error."""
    ref = oracle.collapsed(w.dtype, A, B, b_col_major=w.b_col_major, fma=False, rows=rows, threads=threads)
    if w.dtype == "i8":
        assert C_gpu_rows.dtype == np.int32
        bad = int((C_gpu_rows != ref).sum())
        assert bad == 0, "%d of %d int32 outputs differ" % (bad, ref.size)
        return 0.0
    S, _ = oracle.abs_sum_rows(w.dtype, A, B, b_col_major=w.b_col_major, rows=rows, threads=threads)
    err = np.abs(C_gpu_rows.astype(np.float64) - ref.astype(np.float64))
    ok = err <= TOL[w.dtype] * S
    assert ok.all(), "max |dC|/S = %g (tolerance %g)" % (float((err / np.maximum(S, 1e-300)).max()), TOL[w.dtype])
    if expect_bit_exact_fma:
        ref1 = oracle.collapsed(w.dtype, A, B, b_col_major=w.b_col_major, fma=True, rows=rows, threads=threads)
        assert C_gpu_rows.tobytes() == ref1.tobytes(), "not bit-identical to the fused-multiply-add chain"
    return float((err / np.maximum(S, 1e-300)).max())


def check_workload(w, threads=8, rows_per_problem=None, fixed_k_order=None):
    """Full element-by-element parity (or on sampled rows when ``rows_per_problem`` is given)."""
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B, fixed_k_order)
    fixed = w.fixed_k_order if fixed_k_order is None else fixed_k_order
    exact = w.dtype == "f32" and fixed
    worst = 0.0
    problems = range(w.batch) if w.batch > 1 else [None]
    for b in problems:
        Ab, Bb, Cb = (A, B, C) if b is None else (A[b], B[b], C[b])
        assert Cb.shape == (w.M, w.N)
        if rows_per_problem is None:
            rows = np.arange(w.M)
        else:
            rng = np.random.default_rng(1234 + (b or 0))
            # sampled rows, always including the first and last row of the problem and of a tile
            fixed_rows = [r for r in (0, 127, 128, 255, 256, 383, 384, 511, 512, w.M - 129, w.M - 1) if 0 <= r < w.M]
            rows = np.unique(np.concatenate([fixed_rows, rng.integers(0, w.M, size=rows_per_problem)]))
        worst = max(worst, compare_rows(w, Ab, Bb, Cb[rows], rows, threads, exact))
    return worst
