"""FlashAttention-2 recurrence on the GPU against the fp64 oracle on the same seeded bf16 operands.

Tolerance: ``|O - O_oracle| <= 4e-3 * A`` element by element, ``A_ic = sum_j softmax_ij |V_jc|``.  The only rounding
of that order on the GPU is the bf16 rounding of the exponentials before the second product (relative 2^-9 = 1.95e-3 per
term, hence at most 1.95e-3 * A in the output); score accumulation, running maximum, normaliser and output are fp32.
"""
import numpy as np
import pytest

from oracle import fa2 as ofa2
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu
AW = inputs.AttentionWorkload
TOL = 4e-3


def gpu_attention(Q, K, V):
    import torch
    from paper_2511_09987_b200 import binding
    dQ, dK, dV = (torch.from_numpy(np.ascontiguousarray(x)).view(torch.bfloat16).cuda() for x in (Q, K, V))
    O = binding.flash_attention(dQ, dK, dV)
    assert binding.last_device_status() == binding.CYC_OK
    torch.cuda.synchronize()
    return O.cpu().numpy()


def check_rows(O_rows, Q_rows, K, V, threads=8):
    ref, _, _, A = ofa2.attention(Q_rows, K, V, 128, threads=threads, with_state=True)
    err = np.abs(O_rows.astype(np.float64) - ref)
    assert np.isfinite(O_rows).all()
    assert (err <= TOL * A + 1e-30).all(), "max error %g of A (tolerance %g)" % (float((err / A).max()), TOL)
    return float((err / A).max())


CASES = [
    AW("one", 1, 1, 1, 64, seed=40),
    AW("one_tile_d128", 1, 128, 128, 128, seed=41),
    AW("a1", 2, 300, 500, 64, seed=20),
    AW("ragged_d128", 3, 129, 257, 128, seed=42),
    AW("single_key", 2, 70, 1, 128, seed=43),
    AW("single_query_many_keys", 1, 1, 1000, 64, seed=44),
    AW("peaked_scores", 2, 256, 640, 128, seed=45, qk_std=3.0),
    AW("flat_scores", 1, 200, 384, 64, seed=46, qk_std=0.05),
    AW("several_tiles", 2, 1000, 2000, 64, seed=47),
    AW("many_problems", 40, 130, 140, 128, seed=48),
    # the grid's last round cut by key range (units = batch * ceil(N / 256); parts of at least two key tiles each)
    AW("tail_after_a_full_round", 150, 256, 1024, 64, seed=49),       # 150 units on 148 SMs: 2 left over, 4 parts each
    AW("three_parts_ragged", 5, 300, 800, 128, seed=51),              # 10 units, 7 key tiles: 3 parts of 2, 2 and 3 tiles
    AW("two_parts_peaked", 37, 512, 640, 128, seed=52, qk_std=3.0),   # 74 units, 2 parts; maxima differ between parts
    AW("tail_second_query_tile_empty", 3, 100, 1500, 64, seed=53),    # 3 units whose second query tile holds no rows
]


@pytest.mark.parametrize("w", CASES, ids=[c.name for c in CASES])
def test_against_the_oracle(w):
    Q, K, V = inputs.make_attention_operands(w)
    O = gpu_attention(Q, K, V)
    assert O.shape == (w.batch, w.N, w.d) and O.dtype == np.float32
    # a long batch: the first problems, a few in the middle and the last ones (which hold the units of the last round)
    problems = range(w.batch) if w.batch <= 48 else sorted(set(range(3)) | set(range(w.batch // 2, w.batch // 2 + 3)) | set(range(w.batch - 8, w.batch)))
    for b in problems:
        check_rows(O[b], Q[b], K[b], V[b])


def test_exact_and_closed_form_cases():
    w = AW("p", 2, 100, 300, 64, seed=50)
    Q, K, V = inputs.make_attention_operands(w)
    # a single key: the output is that key's value row, exactly
    O = gpu_attention(Q, K[:, :1], V[:, :1])
    vrow = inputs.bf16_bits_to_f32(V[:, :1])
    assert (O == np.broadcast_to(vrow, O.shape)).all()
    # zero queries: all weights equal, the output is the column mean of V
    O = gpu_attention(np.zeros_like(Q), K, V)
    mean = inputs.bf16_bits_to_f32(V).astype(np.float64).mean(axis=1, keepdims=True)
    assert np.abs(O - mean).max() <= 1e-6
    # run to run identical
    a, b = gpu_attention(Q, K, V), gpu_attention(Q, K, V)
    assert (a == b).all()


def test_sliced_tail_is_reproducible_and_per_stream():
    """Units cut by key range and folded by whichever part arrives last: the same bits every time, on any stream (each
    stream has its own scratch), and from two streams at once."""
    import torch
    from paper_2511_09987_b200 import binding
    w = AW("parts", 3, 300, 900, 64, seed=54)   # 6 units, 8 key tiles: 4 parts each
    Q, K, V = inputs.make_attention_operands(w)
    first = gpu_attention(Q, K, V)
    for _ in range(5):
        assert (gpu_attention(Q, K, V) == first).all()
    dQ, dK, dV = (torch.from_numpy(np.ascontiguousarray(x)).view(torch.bfloat16).cuda() for x in (Q, K, V))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for rep in range(4):
        for st in (s1, s2):
            with torch.cuda.stream(st):
                outs.append(binding.flash_attention(dQ, dK, dV))
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.CYC_OK
    for o in outs:
        assert (o.cpu().numpy() == first).all()


def test_full_size_every_query_row():
    """a2 at full size: every query row of every problem (all 32 x 4096 x 128 outputs) against the oracle."""
    import os
    w = inputs.ATTENTION_WORKLOADS["a2"]
    Q, K, V = inputs.make_attention_operands(w)
    O = gpu_attention(Q, K, V)
    worst = 0.0
    for b in range(w.batch):
        worst = max(worst, check_rows(O[b], Q[b], K[b], V[b], threads=os.cpu_count() or 8))
    assert worst < TOL


def test_quick_full_size_sampled_rows():
    w = inputs.ATTENTION_WORKLOADS["a2"]
    Q, K, V = inputs.make_attention_operands(w)
    O = gpu_attention(Q, K, V)
    rows = np.array([0, 1, 31, 32, 127, 128, 129, 1000, 2047, 2048, 3000, 4094, 4095])
    worst = 0.0
    for b in (0, 1, 7, 16, 31):
        worst = max(worst, check_rows(O[b][rows], Q[b][rows], K[b], V[b], threads=12))
    assert worst < TOL
