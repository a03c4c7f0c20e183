"""Behaviour of the library around the kernels: the dispatch log, the descriptor cache, and calls captured into CUDA
graphs (which must not allocate: a stream without sliced-tail scratch runs the plain schedule while it is captured)."""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import fa2 as ofa2
from paper_2511_09987_b200 import inputs

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_dispatch_log_names_every_kernel_selection():
    code = (
        "import torch\n"
        "from paper_2511_09987_b200 import binding\n"
        "a = torch.randn(384, 256, device='cuda').to(torch.bfloat16); b = torch.randn(256, 512, device='cuda').to(torch.bfloat16)\n"
        "binding.recurrence_matmul(a, b)\n"
        "q = torch.randn(2, 300, 64, device='cuda').to(torch.bfloat16); k = torch.randn(2, 900, 64, device='cuda').to(torch.bfloat16)\n"
        "binding.flash_attention(q, k, k)\n"
        "torch.cuda.synchronize()\n"
    )
    for flag, expect in (("1", True), ("0", False), (None, False)):
        env = dict(os.environ, PYTHONPATH=ROOT)
        env.pop("CYC_LOG", None)
        if flag is not None:
            env["CYC_LOG"] = flag
        out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
        assert out.returncode == 0, out.stderr
        lines = [l for l in out.stderr.splitlines() if l.startswith("cyc:")]
        if expect:
            assert any("M=384 N=512 K=256" in l and l.endswith("-> tcgen05_pair") for l in lines), lines
            assert any("attention batch=2 N=300 M=900 d=64" in l and "tail_parts=" in l for l in lines), lines
        else:
            assert not lines


def test_descriptor_cache_tells_buffers_and_shapes_apart():
    import torch
    from paper_2511_09987_b200 import binding
    g = torch.Generator(device="cuda").manual_seed(3)
    def operands(M, N, K):
        return (torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16), torch.randn((K, N), device="cuda", generator=g).to(torch.bfloat16))
    sets = [operands(256, 256, 256), operands(256, 256, 256), operands(384, 256, 256), operands(256, 384, 128)]
    for _ in range(3):   # the same buffers come back: cached maps must still belong to them
        for a, b in sets:
            c = binding.recurrence_matmul(a, b)
            ref = a.float() @ b.float()
            assert (c - ref).abs().max().item() <= 4e-3 * (a.float().abs() @ b.float().abs()).max().item()
    # a buffer of another shape at an address that was used before
    a, b = sets[0]
    flat = a.reshape(-1)
    a2 = flat[: 128 * 512].reshape(128 * 2, 256)   # same base address, same shape: same map, same result
    assert torch.equal(binding.recurrence_matmul(a2, b), binding.recurrence_matmul(a, b))
    a3 = flat[: 512 * 128].reshape(512, 128)        # same base address, other shape
    b3 = torch.randn((128, 256), device="cuda", generator=g).to(torch.bfloat16)
    c3 = binding.recurrence_matmul(a3, b3)
    assert (c3 - a3.float() @ b3.float()).abs().max().item() <= 4e-3 * (a3.float().abs() @ b3.float().abs()).max().item()


def test_attention_captured_into_a_graph_on_a_fresh_stream():
    """While a stream is being captured the library must not allocate: with no scratch for that stream yet the launch
    runs without the sliced tail, and the replayed graph gives the result of the eager call."""
    import torch
    from paper_2511_09987_b200 import binding
    w = inputs.AttentionWorkload("g", 3, 300, 900, 64, seed=60)
    Q, K, V = inputs.make_attention_operands(w)
    dQ, dK, dV = (torch.from_numpy(np.ascontiguousarray(x)).view(torch.bfloat16).cuda() for x in (Q, K, V))
    eager = binding.flash_attention(dQ, dK, dV)
    torch.cuda.synchronize()
    out = torch.empty_like(eager)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):   # an allocation by the library here would make the capture fail
        binding.flash_attention(dQ, dK, dV, out)
    out.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.CYC_OK
    o = out.cpu().numpy()
    for b in range(w.batch):
        ref, _, _, Aw = ofa2.attention(Q[b], K[b], V[b], 128, threads=4, with_state=True)
        assert (np.abs(o[b] - ref) <= 4e-3 * Aw + 1e-30).all()
    # (the eager call above ran the sliced schedule: its parts round their exponentials against other reference maxima,
    # so the two results agree to the bf16 rounding of the exponentials, not bit for bit -- both are within tolerance)
    e = eager.cpu().numpy()
    for b in range(w.batch):
        ref, _, _, Aw = ofa2.attention(Q[b], K[b], V[b], 128, threads=4, with_state=True)
        assert (np.abs(e[b] - ref) <= 4e-3 * Aw + 1e-30).all()
