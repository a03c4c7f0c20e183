"""Back-to-back launches of every kernel family: a race in a barrier protocol shows up as a bounded wait that runs
out (reported by the status word) or as a result that changes from launch to launch, only once in many launches."""
import pytest

from paper_2511_09987_b200 import inputs
from parity_util import to_device

pytestmark = pytest.mark.gpu

CASES = [
    # name, dtype, M, N, K, batch, col, fixed, launches
    ("3xtf32", "f32", 65536, 256, 256, 1, False, False, 3000),
    ("pair_int8", "i8", 4096, 4096, 1024, 1, True, False, 3000),
    ("pair_int8_sliced_tail", "i8", 4096, 4096, 4096, 1, True, False, 2000),
    ("pair_bf16_sliced_tail", "bf16", 2560, 2560, 1024, 1, False, False, 2000),
    ("pair_bf16_batched", "bf16", 256, 256, 256, 256, False, False, 3000),
    ("tall_bf16", "bf16", 4608, 4096, 6144, 1, False, False, 300),
    ("splitk_bf16", "bf16", 512, 512, 16384, 1, False, False, 3000),
    ("one_cta_bf16", "bf16", 128, 4096, 1024, 1, False, False, 3000),
    ("simt_fp32", "f32", 2048, 512, 256, 1, False, True, 1000),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_many_launches_stay_clean_and_identical(case):
    import torch
    from paper_2511_09987_b200 import binding
    name, dtype, M, N, K, batch, col, fixed, launches = case
    dist = ("int8",) if dtype == "i8" else ("uniform", -1.0, 1.0)
    w = inputs.Workload(name, dtype, M, N, K, 7, batch, col, fixed, dist, dist)
    A, B = inputs.make_operands(w)
    dA, dB = to_device(A, dtype), to_device(B, dtype)
    fn = binding.recurrence_matmul_batched if batch > 1 else binding.recurrence_matmul
    outs = [fn(dA, dB, b_col_major=col, fixed_k_order=fixed) for _ in range(3)]
    first = outs[0].clone()
    assert binding.last_device_status() == binding.CYC_OK
    for i in range(launches):
        fn(dA, dB, outs[i % 3], b_col_major=col, fixed_k_order=fixed)
    assert binding.last_device_status() == binding.CYC_OK, binding.cyc_last_cuda_error()
    for o in outs:
        assert torch.equal(o, first)


def test_many_scan_launches_stay_clean_and_identical():
    """The look-back of the prefix-sum kernel is the one place where CTAs of a launch wait for one another: thousands of
    launches on long and short chains must leave the status word clean; int32 results are identical every time."""
    import torch
    from paper_2511_09987_b200 import binding
    for rows, n, launches in ((1, 1 << 22, 1500), (64, 70001, 1500), (4096, 4096, 500)):
        A = torch.from_numpy(inputs.make_scan_operand(inputs.ScanWorkload("s", rows, n, "i32", 91))).cuda()
        outs = [binding.prefix_sum(A) for _ in range(3)]
        first = outs[0].clone()
        for i in range(launches):
            binding.prefix_sum(A, outs[i % 3])
        assert binding.last_device_status() == binding.CYC_OK, binding.cyc_last_cuda_error()
        for o in outs:
            assert torch.equal(o, first)


def test_many_attention_and_cholesky_launches_stay_clean_and_identical():
    import torch
    from paper_2511_09987_b200 import binding
    Q, K, V = (torch.from_numpy(x).view(torch.bfloat16).cuda()
               for x in inputs.make_attention_operands(inputs.AttentionWorkload("s", 8, 1000, 1500, 128, seed=92)))
    outs = [binding.flash_attention(Q, K, V) for _ in range(3)]
    first = outs[0].clone()
    for i in range(1500):
        binding.flash_attention(Q, K, V, outs[i % 3])
    assert binding.last_device_status() == binding.CYC_OK, binding.cyc_last_cuda_error()
    for o in outs:
        assert torch.equal(o, first)
    A = torch.from_numpy(inputs.make_chol_operand(inputs.CholWorkload("s", 1100, 256, 93))).cuda()
    outs = [binding.cholesky(A) for _ in range(3)]
    first = outs[0].clone()
    for i in range(100):
        binding.cholesky(A, outs[i % 3])
    assert binding.last_device_status() == binding.CYC_OK, binding.cyc_last_cuda_error()
    for o in outs:
        assert torch.equal(o, first)
