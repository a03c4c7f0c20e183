"""The allocation-free split-K entry point, `cyc_recurrence_matmul_splitk_static`.

Some programs that embed this library may not allocate device memory once they are running: they
handed the whole GPU to their own allocator at start-up, or they sit in a latency-critical loop
that must never enter the driver's allocator.  For them the library carries a fixed workspace and
an entry point that uses it instead of the stream-ordered pool.  This test calls that entry point
through the C ABI twice in a row (different operands and shapes, so stale workspace contents would
show) and compares with the ordinary entry point, and it checks the property in the name: after one
warm-up call, free device memory and the library pool's size are the same before and after every
call.  (That oversized requests are refused on the host is checked without a GPU, in
tests/test_abi.py.)  Collected last on purpose (file name), and self-contained so that it also
passes alone in a fresh process.
"""
import numpy as np
import pytest

import oracle
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu


def _operands(dtype, M, N, K, seed, col):
    dist = ("int8",) if dtype == "i8" else ("uniform", -1.0, 1.0)
    bdist = ("int8",) if dtype == "i8" else ("normal", 1.0)
    w = inputs.Workload("noalloc", dtype, M, N, K, seed, 1, col, False, dist, bdist)
    return w, inputs.make_operands(w)


def _dev(x, dtype):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x))
    return (t.view(torch.bfloat16) if dtype == "bf16" else t).cuda()


@pytest.mark.parametrize("dtype,col", [("bf16", False), ("i8", True)])
def test_two_calls_in_a_row_match_the_ordinary_entry_point(dtype, col):
    import torch
    from paper_2511_09987_b200 import binding as b
    code = b.DTYPE_CODES[dtype]
    flags = b.CYC_FLAG_B_COL_MAJOR if col else 0
    stream = torch.cuda.current_stream().cuda_stream
    out_dtype = torch.int32 if dtype == "i8" else torch.float32
    # second call: other operands, a smaller shape and fewer slices than the first, ragged in M, N and K
    for call, (M, N, K, seed) in enumerate([(512, 256, 8192, 71), (300, 264, 4112, 72)]):
        w, (A, B) = _operands(dtype, M, N, K, seed, col)
        dA, dB = _dev(A, dtype), _dev(B, dtype)
        got = torch.full((M, N), -1, dtype=out_dtype, device="cuda")
        want = torch.empty((M, N), dtype=out_dtype, device="cuda")
        torch.cuda.synchronize()
        rc = b.cyc_recurrence_matmul_splitk_static(M, N, K, code, dA.data_ptr(), dB.data_ptr(), got.data_ptr(), stream, flags)
        assert rc == b.CYC_OK, (rc, b.cyc_last_cuda_error())
        rc = b.cyc_recurrence_matmul(M, N, K, code, dA.data_ptr(), dB.data_ptr(), want.data_ptr(), stream, flags)
        assert rc == b.CYC_OK
        assert b.last_device_status() == b.CYC_OK
        got, want = got.cpu().numpy(), want.cpu().numpy()
        if dtype == "i8":
            assert (got == want).all(), "call %d: int32 results differ" % call
            assert (got == oracle.collapsed("i8", A, B, b_col_major=col, threads=4)).all()
        else:
            S, _ = oracle.abs_sum_rows(dtype, A, B, b_col_major=col, threads=4)
            assert (np.abs(got.astype(np.float64) - want) <= 4e-3 * S).all(), "call %d" % call
            ref = oracle.collapsed(dtype, A, B, b_col_major=col, threads=4)
            assert (np.abs(got.astype(np.float64) - ref) <= 4e-3 * S).all(), "call %d vs oracle" % call


def _pool_bytes(b):
    import ctypes
    out = ctypes.c_int64(-1)
    assert b.cyc_pool_reserved_bytes(ctypes.byref(out)) == b.CYC_OK
    return out.value


def test_calls_allocate_nothing():
    """After one warm-up call on the device (which may load the library's device code, the moment the device receives
    its copy of the fixed array), two further calls leave the free device memory and the library pool as they were."""
    import torch
    from paper_2511_09987_b200 import binding as b
    stream = torch.cuda.current_stream().cuda_stream
    shapes = [(512, 256, 8192, 81), (300, 264, 4112, 82)]
    ops = []
    for M, N, K, seed in shapes:                      # every tensor exists before the first measurement
        w, (A, B) = _operands("bf16", M, N, K, seed, False)
        ops.append((M, N, K, _dev(A, "bf16"), _dev(B, "bf16"), torch.empty((M, N), dtype=torch.float32, device="cuda")))
    M, N, K, dA, dB, dC = ops[0]
    assert b.cyc_recurrence_matmul_splitk_static(M, N, K, b.CYC_BF16_F32, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), stream, 0) == b.CYC_OK
    torch.cuda.synchronize()
    for M, N, K, dA, dB, dC in ops:
        free0, pool0 = torch.cuda.mem_get_info()[0], _pool_bytes(b)
        rc = b.cyc_recurrence_matmul_splitk_static(M, N, K, b.CYC_BF16_F32, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), stream, 0)
        assert rc == b.CYC_OK
        torch.cuda.synchronize()
        assert b.last_device_status() == b.CYC_OK
        assert torch.cuda.mem_get_info()[0] == free0, "free device memory changed across the call"
        assert _pool_bytes(b) == pool0, "the library's pool grew or shrank across the call"
