"""The seeded operand generator: published test vector, determinism, ranges,
moments and bf16 rounding."""
import numpy as np

from paper_2511_09987_b200 import inputs


def test_splitmix64_published_vector():
    # splitmix64 seeded with 0: the first three outputs of the published reference implementation
    z = inputs._bits(0, 0, 0, 3)
    assert [int(x) for x in z] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_counter_based_and_deterministic():
    a = inputs.uniform_f32(3, 0, 1000, -1.0, 1.0)
    b = inputs.uniform_f32(3, 0, 1000, -1.0, 1.0)
    assert a.tobytes() == b.tobytes()
    big = inputs.uniform_f32(3, 0, inputs._CHUNK + 17, -1.0, 1.0)   # crosses a chunk boundary
    assert big[:1000].tobytes() == a.tobytes()
    assert inputs.uniform_f32(4, 0, 1000, -1.0, 1.0).tobytes() != a.tobytes()
    assert inputs.uniform_f32(3, 1, 1000, -1.0, 1.0).tobytes() != a.tobytes()


def test_distributions():
    n = 1 << 18
    u = inputs.uniform_f32(1, 0, n, -2.0, 2.0).astype(np.float64)
    assert u.min() >= -2.0 and u.max() < 2.0
    assert abs(u.mean()) < 0.02 and abs(u.std() - 4.0 / np.sqrt(12.0)) < 0.02
    g = inputs.normal_f32(1, 1, n, 0.1).astype(np.float64)
    assert abs(g.mean()) < 0.002 and abs(g.std() - 0.1) < 0.002 and np.isfinite(g).all()
    assert abs((np.abs(g) < 0.1).mean() - 0.6827) < 0.01
    i = inputs.uniform_i8(1, 0, n)
    assert i.dtype == np.int8 and i.min() == -128 and i.max() == 127
    counts = np.bincount(i.astype(np.int64) + 128, minlength=256)
    assert counts.min() > 0.8 * n / 256 and counts.max() < 1.2 * n / 256


def test_bf16_rounding_ties_to_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -3.14159, 0.0], np.float32)
    h = inputs.f32_to_bf16_bits(x)
    back = inputs.bf16_bits_to_f32(h).astype(np.float64)
    assert back.tolist() == [1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -3.140625, 0.0]


def test_workload_table():
    w = inputs.WORKLOADS
    assert (w["c1"].M, w["c1"].N, w["c1"].K, w["c1"].dtype, w["c1"].seed) == (64, 64, 64, "f32", 0)
    assert (w["c2"].M, w["c2"].dtype, w["c2"].b_col_major, w["c2"].seed) == (4096, "i8", True, 1)
    assert (w["c3"].M, w["c3"].dtype, w["c3"].seed) == (8192, "bf16", 2)
    assert (w["c4"].M, w["c4"].N, w["c4"].K, w["c4"].seed) == (65536, 256, 256, 3)
    assert (w["c5"].batch, w["c5"].M, w["c5"].seed) == (1024, 256, 4)
    assert w["c3"].algorithmic_bytes == 536870912 and w["c5"].algorithmic_bytes == 536870912
    assert w["c2"].algorithmic_bytes == 100663296 and w["c4"].algorithmic_bytes == 134479872
    s = inputs.scaled(w["c5"], batch=2, M=4, N=5, K=6)
    A, B = inputs.make_operands(s)
    assert A.shape == (2, 4, 6) and B.shape == (2, 6, 5) and A.dtype == np.uint16
    s = inputs.scaled(w["c2"], M=4, N=5, K=6)
    A, B = inputs.make_operands(s)
    assert A.shape == (4, 6) and B.shape == (5, 6) and A.dtype == np.int8
