"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded operands.  int8 must be bit-exact; fp32 within 1e-5 * S and bf16
within 4e-3 * S, S_ij = sum_k |A_ik||B_kj|; the strict fp32 path must reproduce the
fused-multiply-add chain bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2511_09987_b200 import inputs
from parity_util import check_workload, gpu_run, to_device

pytestmark = pytest.mark.gpu

W = inputs.WORKLOADS


def wl(dtype, M, N, K, seed, batch=1, col=False, fixed=False):
    if dtype == "i8":
        return inputs.Workload("t", "i8", M, N, K, seed, batch, col, fixed, ("int8",), ("int8",))
    return inputs.Workload("t", dtype, M, N, K, seed, batch, col, fixed, ("uniform", -1.0, 1.0), ("normal", 1.0))


def family(w):
    from paper_2511_09987_b200 import binding
    return binding.kernel_for(w.batch, w.M, w.N, w.K, w.dtype, b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)


# ------------------------------------------------------------------ general (SIMT) kernel
@pytest.mark.parametrize("shape", [(1, 1, 1), (64, 64, 64), (130, 70, 37), (257, 129, 513), (5, 300, 1), (128, 128, 16),
                                   (256, 256, 64), (31, 1, 100)])
@pytest.mark.parametrize("col", [False, True])
def test_simt_fp32_strict_order_bit_exact(shape, col):
    w = wl("f32", *shape, seed=11, col=col, fixed=True)
    assert family(w) == "simt"
    check_workload(w)   # includes the bit-for-bit comparison with the fused chain


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
@pytest.mark.parametrize("shape", [(1, 1, 1), (65, 127, 33), (200, 131, 77), (3, 5, 300)])
@pytest.mark.parametrize("col", [False, True])
def test_simt_unaligned_shapes(dtype, shape, col):
    w = wl(dtype, *shape, seed=12, col=col)
    assert family(w) == "simt"
    A, B = inputs.make_operands(w)
    C = gpu_run(w, A, B)
    ref = oracle.collapsed(dtype, A, B, b_col_major=col)
    assert C.tobytes() == ref.tobytes()   # a strict chain of exact products: identical in both types


def test_simt_batched_fp32():
    w = wl("f32", 70, 40, 50, seed=13, batch=4, fixed=True)
    check_workload(w)


def test_config_c1():
    assert family(W["c1"]) == "simt"
    worst = check_workload(W["c1"])
    assert worst < 1e-5


# ------------------------------------------------------------------ tensor-core kernel, small and ragged
UMMA_SHAPES = [(128, 128, 64), (128, 256, 64), (128, 256, 128), (256, 512, 256), (256, 256, 1024), (300, 520, 200),
               (129, 264, 72), (200, 96, 136), (1, 8, 8), (127, 392, 520)]


@pytest.mark.parametrize("shape", UMMA_SHAPES)
@pytest.mark.parametrize("col", [False, True])
def test_umma_bf16(shape, col):
    w = wl("bf16", *shape, seed=21, col=col)
    assert family(w).startswith("tcgen05")
    check_workload(w)


@pytest.mark.parametrize("shape", [(128, 256, 128), (128, 128, 128), (384, 528, 400), (256, 256, 2048), (130, 272, 144),
                                   (1, 16, 16), (250, 112, 1040)])
@pytest.mark.parametrize("col", [True, False])
def test_umma_int8_bit_exact(shape, col):
    w = wl("i8", *shape, seed=22, col=col)
    assert family(w).startswith("tcgen05")
    check_workload(w)


@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 520, 200), (129, 264, 72), (512, 384, 36), (1000, 260, 1028)])
@pytest.mark.parametrize("col", [False, True])
def test_fp32_split_tf32_on_tensor_cores(shape, col):
    w = wl("f32", *shape, seed=41, col=col, fixed=False)
    assert family(w) == "tcgen05_3xtf32"
    worst = check_workload(w)          # 1e-5 * S
    assert worst < 2e-6                # the split leaves about 2^-21 per product


@pytest.mark.parametrize("shape", [(18944, 256, 256), (20001, 256, 256), (19000, 200, 256), (19500, 132, 100), (18944, 256, 32),
                                   (30000, 252, 36), (19000, 128, 256), (21000, 64, 96), (19001, 100, 4), (19000, 4, 256), (19000, 20, 8)])
@pytest.mark.parametrize("col", [False, True])
def test_fp32_weight_stationary_on_tensor_cores(shape, col):
    """Small B under a long A: B^T split once and kept in tensor memory / shared memory, A streamed in 128-row tiles
    (ragged last tile, ragged n and k included; B stored [K][N] or [N][K])."""
    if col and shape[2] % 4:
        pytest.skip("row pitch of B stored [N][K] not a multiple of 16 bytes")
    w = wl("f32", *shape, seed=43, col=col, fixed=False)
    assert family(w) == "tcgen05_3xtf32_ws"
    worst = check_workload(w, rows_per_problem=600)
    assert worst < 2e-6


def test_fp32_weight_stationary_closed_forms():
    import torch
    from paper_2511_09987_b200 import binding
    M, n = 19200, 256
    assert binding.kernel_for(1, M, n, n, "f32") == "tcgen05_3xtf32_ws"
    X = (torch.randn(M, n, device="cuda") * 3).float()
    I = torch.eye(n, device="cuda")
    out = binding.recurrence_matmul(X, I)                      # B = I returns A to within 2^-21 relative
    assert (out - X).abs().max().item() <= 2.0 ** -21 * X.abs().max().item()
    Xi = torch.randint(-1000, 1000, (M, n), device="cuda").float()      # 11-bit integers: hi part exact, lo zero
    assert torch.equal(binding.recurrence_matmul(Xi, I), Xi)
    P = torch.eye(n, device="cuda")[torch.randperm(n, device="cuda")]   # a permutation of the columns, exactly
    assert torch.equal(binding.recurrence_matmul(Xi, P), Xi @ P)
    ones = torch.ones((M, n), device="cuda")
    assert (binding.recurrence_matmul(ones, torch.ones((n, n), device="cuda")) == n).all().item()
    assert binding.last_device_status() == binding.CYC_OK


def test_fp32_weight_stationary_non_finite_values_stay_in_their_rows_and_columns():
    import torch
    from paper_2511_09987_b200 import binding
    M, n, k = 19072, 256, 256
    g = torch.Generator(device="cuda").manual_seed(5)
    A = torch.rand((M, k), device="cuda", generator=g) + 0.5          # positive: no 0 * inf
    B = torch.rand((k, n), device="cuda", generator=g) + 0.5
    A[5, 7] = float("inf"); A[9000, 3] = float("nan"); A[M - 1, k - 1] = float("-inf")
    B[17, 200] = float("inf")
    assert binding.kernel_for(1, M, n, k, "f32") == "tcgen05_3xtf32_ws"
    C = binding.recurrence_matmul(A, B)
    ref = A.double() @ B.double()
    # Where the exact result is not finite the split arithmetic may give inf or NaN (an infinite hi part meets a lo part
    # that happens to be exactly zero): what must hold is that every such entry is non-finite, every other entry is
    # finite and as accurate as ever, and a row of infinities has the right sign where the exact result has one.
    fin = torch.isfinite(ref)
    assert torch.equal(torch.isfinite(C), fin)
    assert (fin.sum(dim=1) == 0).sum().item() == 3 and (fin.sum(dim=0) == 0).sum().item() == 1   # three rows, one column
    assert ((C.double() - ref).abs()[fin] <= 1e-5 * (A.double().abs() @ B.double().abs())[fin]).all().item()
    both_inf = torch.isinf(C) & torch.isinf(ref)
    assert torch.equal(torch.sign(C[both_inf]).double(), torch.sign(ref[both_inf]))
    assert torch.isnan(C[9000]).all().item()
    assert binding.last_device_status() == binding.CYC_OK


def test_fp32_split_closed_forms():
    import torch
    from paper_2511_09987_b200 import binding
    n = 384
    X = (torch.randn(n, n, device="cuda") * 3).float()
    I = torch.eye(n, device="cuda")
    assert binding.kernel_for(1, n, n, n, "f32") == "tcgen05_3xtf32"
    # hi + lo carries 22 of the 24 significand bits, so A = I returns B to within 2^-21 relative
    out = binding.recurrence_matmul(I, X)
    assert (out - X).abs().max().item() <= 2.0 ** -21 * X.abs().max().item()
    ones = torch.ones((n, n), device="cuda")
    assert (binding.recurrence_matmul(ones, ones) == n).all().item()
    Xi = torch.randint(-1000, 1000, (n, n), device="cuda").float()      # 11-bit integers: hi part exact, lo zero
    assert torch.equal(binding.recurrence_matmul(I, Xi), Xi)


def test_umma_int8_extreme_values():
    import torch
    from paper_2511_09987_b200 import binding
    K = 4096
    A = torch.full((128, K), -128, dtype=torch.int8, device="cuda")
    B = torch.full((256, K), -128, dtype=torch.int8, device="cuda")
    C = binding.recurrence_matmul(A, B, b_col_major=True)
    assert (C == K * 128 * 128).all().item()       # 2^26: every partial sum stays exact
    B.fill_(127)
    assert (binding.recurrence_matmul(A, B, b_col_major=True) == -K * 128 * 127).all().item()


def test_umma_closed_forms_bf16():
    import torch
    from paper_2511_09987_b200 import binding
    n = 384
    X = torch.randint(-64, 64, (n, n), device="cuda").to(torch.bfloat16)
    I = torch.eye(n, device="cuda", dtype=torch.bfloat16)
    perm = torch.randperm(n, device="cuda")
    P = I[perm]
    assert torch.equal(binding.recurrence_matmul(I, X), X.float())            # A = I  =>  C = B
    assert torch.equal(binding.recurrence_matmul(X, I), X.float())            # B = I  =>  C = A
    assert torch.equal(binding.recurrence_matmul(P, X), X.float()[perm])      # row permutation
    assert torch.equal(binding.recurrence_matmul(X, P, b_col_major=True), X.float()[:, perm])   # stored B^T = P
    ones = torch.ones((n, n), device="cuda", dtype=torch.bfloat16)
    assert (binding.recurrence_matmul(ones, ones) == n).all().item()


def test_umma_tall_tiles_ragged():
    # 512 x 256 tiles (long k loop, at least 74 tiles), ragged in every dimension
    w = wl("bf16", 4100, 2600, 6152, seed=51)
    assert family(w) == "tcgen05_pair_tall"
    check_workload(w, rows_per_problem=24)
    w = wl("bf16", 4100, 2600, 6152, seed=52, col=True)
    check_workload(w, rows_per_problem=64)
    w = wl("i8", 4100, 2320, 12304, seed=53, col=True)
    assert family(w) == "tcgen05_pair_tall"
    check_workload(w, rows_per_problem=64)
    w = wl("i8", 4100, 2320, 12304, seed=54, col=False)
    check_workload(w, rows_per_problem=64)
    # batched: 20 problems of 600 x 304 x 6152 -> 2 x 2 tall tiles each
    w = wl("bf16", 600, 304, 6152, seed=55, batch=20)
    assert family(w) == "tcgen05_pair_tall"
    check_workload(w, rows_per_problem=24)


@pytest.mark.parametrize("case", [("bf16", 256, 256, 8192, False, 1), ("i8", 512, 256, 16400, True, 1), ("bf16", 300, 264, 4104, False, 1),
                                  ("bf16", 300, 264, 4104, True, 1), ("i8", 260, 130, 4096, True, 1), ("bf16", 256, 256, 2048, False, 3),
                                  ("i8", 384, 272, 8192, False, 2)])
def test_split_k_few_tiles_long_k(case):
    dtype, M, N, K, col, batch = case
    w = wl(dtype, M, N, K, seed=61, col=col, batch=batch)
    assert family(w) == "tcgen05_pair_splitk"
    check_workload(w)
    A, B = inputs.make_operands(w)
    assert gpu_run(w, A, B).tobytes() == gpu_run(w, A, B).tobytes()      # slices are added in a fixed order
    # with the fixed-order flag one CTA pair owns each output for the whole k loop
    wf = wl(dtype, M, N, K, seed=61, col=col, batch=batch, fixed=True)
    assert family(wf) == "tcgen05_pair"
    check_workload(wf)


def test_umma_many_tiles_per_cta():
    # 512 tiles on 148 SMs: every CTA walks 3-4 tiles, both TMEM accumulators and both barrier phases
    check_workload(wl("bf16", 4096, 4096, 64, seed=23), rows_per_problem=96)
    check_workload(wl("i8", 4096, 4096, 128, seed=24, col=True), rows_per_problem=96)


@pytest.mark.parametrize("dtype,col", [("bf16", False), ("bf16", True), ("i8", True)])
def test_umma_batched(dtype, col):
    check_workload(wl(dtype, 256, 256, 256, seed=25, batch=5, col=col))
    check_workload(wl(dtype, 130, 136, 80, seed=26, batch=3, col=col))


def test_batched_with_padding_strides():
    import torch
    from paper_2511_09987_b200 import binding
    w = wl("bf16", 128, 136, 72, seed=27, batch=3)
    A, B = inputs.make_operands(w)
    pad = 64
    dA = torch.zeros((3, 128 * 72 + pad), dtype=torch.bfloat16, device="cuda")
    dB = torch.zeros((3, 72 * 136 + pad), dtype=torch.bfloat16, device="cuda")
    dC = torch.full((3, 128 * 136 + pad), -7.0, dtype=torch.float32, device="cuda")
    dA[:, :128 * 72] = to_device(A, "bf16").reshape(3, -1)
    dB[:, :72 * 136] = to_device(B, "bf16").reshape(3, -1)
    binding.check(binding.cyc_recurrence_matmul_batched(3, 128, 136, 72, binding.CYC_BF16_F32, dA.data_ptr(), dA.shape[1],
                                                        dB.data_ptr(), dB.shape[1], dC.data_ptr(), dC.shape[1],
                                                        torch.cuda.current_stream().cuda_stream, 0))
    torch.cuda.synchronize()
    out = dC.cpu().numpy()
    assert (out[:, 128 * 136:] == -7.0).all()     # padding untouched
    ref = oracle.batched_collapsed("bf16", A, B)
    S = np.stack([oracle.abs_sum_rows("bf16", A[b], B[b])[0] for b in range(3)])
    assert (np.abs(out[:, :128 * 136].reshape(3, 128, 136) - ref) <= 4e-3 * S).all()


def test_results_are_reproducible():
    for w in (wl("bf16", 512, 512, 512, seed=28), wl("f32", 300, 200, 100, seed=29, fixed=True)):
        A, B = inputs.make_operands(w)
        assert gpu_run(w, A, B).tobytes() == gpu_run(w, A, B).tobytes()


def test_output_rows_outside_problem_untouched():
    import torch
    from paper_2511_09987_b200 import binding
    # C is exactly M*N: a guard region after it must stay intact for ragged tiles
    for dtype, M, N, K in (("bf16", 130, 264, 72), ("f32", 130, 70, 37)):
        w = wl(dtype, M, N, K, seed=30, fixed=(dtype == "f32"))
        A, B = inputs.make_operands(w)
        buf = torch.full((M * N + 4096,), 123.0, dtype=torch.float32, device="cuda")
        binding.recurrence_matmul(to_device(A, dtype), to_device(B, dtype), buf[:M * N].view(M, N), fixed_k_order=w.fixed_k_order)
        torch.cuda.synchronize()
        assert (buf[M * N:] == 123.0).all().item()


def test_host_entry_point():
    import torch
    from paper_2511_09987_b200 import binding
    w = wl("bf16", 256, 256, 128, seed=31, batch=2)
    A, B = inputs.make_operands(w)
    hA = torch.from_numpy(A).view(torch.bfloat16).pin_memory()
    hB = torch.from_numpy(B).view(torch.bfloat16).pin_memory()
    hC = torch.empty((2, 256, 256), dtype=torch.float32).pin_memory()
    binding.recurrence_matmul_host(hA, hB, hC)
    assert hC.numpy().tobytes() == gpu_run(w, A, B).tobytes()


@pytest.mark.parametrize("case", [("bf16", 3000, 1024, 2048, 1, False), ("i8", 256, 256, 1024, 40, True), ("f32", 2500, 512, 1024, 1, False)])
def test_host_entry_point_chunked_pipeline(case):
    # large enough (> 16 MB of A and C) for the chunked upload / compute / download pipeline; ragged last chunk
    import torch
    from paper_2511_09987_b200 import binding
    dtype, M, N, K, batch, col = case
    w = wl(dtype, M, N, K, seed=32, batch=batch, col=col)
    A, B = inputs.make_operands(w)
    hA, hB = torch.from_numpy(A), torch.from_numpy(B)
    if dtype == "bf16":
        hA, hB = hA.view(torch.bfloat16), hB.view(torch.bfloat16)
    hA, hB = hA.pin_memory(), hB.pin_memory()
    shape = (batch, M, N) if batch > 1 else (M, N)
    hC = torch.full(shape, 7, dtype=torch.int32 if dtype == "i8" else torch.float32).pin_memory()
    binding.recurrence_matmul_host(hA, hB, hC, b_col_major=col)
    want = gpu_run(w, A, B)
    got = hC.numpy()
    if dtype == "i8":
        assert (got == want).all()
    else:
        # a chunk of rows may be served by another kernel than the whole problem: compare within the tolerance
        prob = range(batch) if batch > 1 else [None]
        for b in prob:
            Ab, Bb, g, wv = (A, B, got, want) if b is None else (A[b], B[b], got[b], want[b])
            rows = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(3).integers(0, M, 40)]))
            S, _ = oracle.abs_sum_rows(dtype, Ab, Bb, b_col_major=col, rows=rows, threads=8)
            tol = 4e-3 if dtype == "bf16" else 1e-5
            assert (np.abs(g[rows].astype(np.float64) - wv[rows]) <= 2 * tol * S).all()
            ref = oracle.collapsed(dtype, Ab, Bb, b_col_major=col, rows=rows, threads=8)
            assert (np.abs(g[rows].astype(np.float64) - ref) <= tol * S).all()


def test_bounded_wait_reports_timeout_and_device_stays_usable():
    # a wait that nothing satisfies runs out of its (short) budget: the kernel returns, the status word says so once,
    # and the next evaluation on the same device is correct
    import torch
    from paper_2511_09987_b200 import binding
    assert binding.last_device_status() == binding.CYC_OK
    stream = torch.cuda.current_stream().cuda_stream
    assert binding.cyc_selftest_bounded_wait(stream, 0) == binding.CYC_ERR_INVALID_ARG
    assert binding.cyc_selftest_bounded_wait(stream, 1 << 30) == binding.CYC_ERR_INVALID_ARG
    assert binding.cyc_selftest_bounded_wait(stream, 100000) == binding.CYC_OK
    assert binding.last_device_status() == binding.CYC_ERR_TIMEOUT
    assert b"wait ran out" in binding.cyc_last_cuda_error()
    assert binding.last_device_status() == binding.CYC_OK          # reported once, then cleared
    check_workload(wl("bf16", 300, 520, 200, seed=33))


def test_two_host_threads_on_two_streams():
    import threading
    import torch
    from paper_2511_09987_b200 import binding
    results, errors = {}, []
    cases = {0: wl("bf16", 512, 512, 512, seed=34), 1: wl("i8", 384, 528, 400, seed=35, col=True)}
    ops = {k: inputs.make_operands(w) for k, w in cases.items()}

    def work(k):
        try:
            w = cases[k]
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                dA, dB = to_device(ops[k][0], w.dtype), to_device(ops[k][1], w.dtype)
                outs = [binding.recurrence_matmul(dA, dB, b_col_major=w.b_col_major) for _ in range(20)]
                s.synchronize()
            results[k] = [o.cpu().numpy() for o in (outs[0], outs[-1])]
        except Exception as exc:  # noqa: BLE001
            errors.append(exc)

    threads = [threading.Thread(target=work, args=(k,)) for k in cases]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for k, w in cases.items():
        ref = oracle.collapsed(w.dtype, ops[k][0], ops[k][1], b_col_major=w.b_col_major, threads=4)
        for got in results[k]:
            if w.dtype == "i8":
                assert (got == ref).all()
            else:
                S, _ = oracle.abs_sum_rows(w.dtype, ops[k][0], ops[k][1], threads=4)
                assert (np.abs(got.astype(np.float64) - ref) <= 4e-3 * S).all()


def test_device_status_is_clean():
    from paper_2511_09987_b200 import binding
    assert binding.last_device_status() == binding.CYC_OK
    assert binding.cyc_launch_count() > 0
