"""Seeded synthetic operands for the recurrence-matmul workloads.

This module only makes input data (host numpy arrays) and describes the five
workload configurations; it contains none of the recurrence's arithmetic.  The
same bytes are handed to the CUDA library and to whatever checks it.

Generator: counter based, so any element can be regenerated independently.
``bits(seed, tensor, index) = splitmix64_finalise(seed * C1 + tensor * C2 + index * GOLDEN)``
with the published splitmix64 finaliser.  From the 64 bits:

* uniform in ``[0,1)``: the top 24 bits times ``2**-24``, mapped to ``[lo,hi)``;
* normal: Box-Muller in float64 from two uniforms taken from the top and the
  bottom 32 bits of the same word (``u1`` shifted into ``(0,1]``), scaled by the
  standard deviation;
* int8: the top byte reinterpreted as a signed byte, uniform on ``[-128,127]``.

bf16 operands are the float32 values rounded to nearest-even and returned as
``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xD1342543DE82EF95)
_C2 = np.uint64(0xA0761D6478BD642F)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22

TENSOR_A = 0
TENSOR_B = 1


def _bits(seed: int, tensor: int, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        z = np.uint64(seed) * _C1 + np.uint64(tensor) * _C2 + (idx + np.uint64(1)) * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def _fill(n: int, fn, dtype) -> np.ndarray:
    out = np.empty(n, dtype=dtype)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        out[s:s + c] = fn(s, c)
    return out


def uniform_f32(seed: int, tensor: int, n: int, lo: float, hi: float) -> np.ndarray:
    def fn(s, c):
        u = (_bits(seed, tensor, s, c) >> np.uint64(40)).astype(np.float64) * 2.0 ** -24
        return (lo + (hi - lo) * u).astype(np.float32)
    return _fill(n, fn, np.float32)


def normal_f32(seed: int, tensor: int, n: int, std: float) -> np.ndarray:
    def fn(s, c):
        z = _bits(seed, tensor, s, c)
        u1 = ((z >> np.uint64(32)).astype(np.float64) + 1.0) * 2.0 ** -32      # (0,1]
        u2 = (z & np.uint64(0xFFFFFFFF)).astype(np.float64) * 2.0 ** -32       # [0,1)
        return (std * np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return _fill(n, fn, np.float32)


def uniform_i8(seed: int, tensor: int, n: int) -> np.ndarray:
    def fn(s, c):
        return (_bits(seed, tensor, s, c) >> np.uint64(56)).astype(np.uint8).view(np.int8)
    return _fill(n, fn, np.int8)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One synthetic configuration.  ``dtype`` is ``"f32"``, ``"bf16"`` or ``"i8"``."""
    name: str
    dtype: str
    M: int
    N: int
    K: int
    seed: int
    batch: int = 1
    b_col_major: bool = False
    fixed_k_order: bool = False
    a_dist: tuple = ("uniform", -1.0, 1.0)
    b_dist: tuple = ("uniform", -1.0, 1.0)

    @property
    def macs(self) -> int:
        return self.batch * self.M * self.N * self.K

    @property
    def in_bytes(self) -> int:
        return {"f32": 4, "bf16": 2, "i8": 1}[self.dtype]

    @property
    def algorithmic_bytes(self) -> int:
        """A and B read once, C written once."""
        return self.batch * ((self.M * self.K + self.K * self.N) * self.in_bytes + self.M * self.N * 4)


WORKLOADS = {
    # fp32 64^3, uniform[-1,1), strict increasing-k accumulation
    "c1": Workload("c1", "f32", 64, 64, 64, seed=0, fixed_k_order=True),
    # int8 x int8 -> int32, 4096^3, A row-major, B column-major
    "c2": Workload("c2", "i8", 4096, 4096, 4096, seed=1, b_col_major=True,
                   a_dist=("int8",), b_dist=("int8",)),
    # bf16 in, fp32 accumulate/out, 8192^3, normal(0,1)
    "c3": Workload("c3", "bf16", 8192, 8192, 8192, seed=2, a_dist=("normal", 1.0), b_dist=("normal", 1.0)),
    # fp32 tall-skinny, A uniform[-1,1), B normal(0, sigma=0.1)
    "c4": Workload("c4", "f32", 65536, 256, 256, seed=3, b_dist=("normal", 0.1)),
    # 1024 independent bf16 problems of 256^3, uniform[-2,2)
    "c5": Workload("c5", "bf16", 256, 256, 256, seed=4, batch=1024,
                   a_dist=("uniform", -2.0, 2.0), b_dist=("uniform", -2.0, 2.0)),
}


def _draw(dist: tuple, dtype: str, seed: int, tensor: int, n: int) -> np.ndarray:
    if dist[0] == "int8":
        if dtype != "i8":
            raise ValueError("int8 distribution needs dtype i8")
        return uniform_i8(seed, tensor, n)
    if dist[0] == "uniform":
        x = uniform_f32(seed, tensor, n, dist[1], dist[2])
    elif dist[0] == "normal":
        x = normal_f32(seed, tensor, n, dist[1])
    else:
        raise ValueError("unknown distribution %r" % (dist,))
    if dtype == "f32":
        return x
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    # small integers for int8 tests drawn from a float distribution are not provided
    raise ValueError("distribution %r not available for dtype %r" % (dist, dtype))


def make_operands(w: Workload):
    """Host arrays ``(A, B)`` for a workload.

    ``A`` has shape ``[batch,] M, K``.  ``B`` has shape ``[batch,] K, N`` or, when
    ``w.b_col_major``, ``[batch,] N, K`` (the element ``B_kj`` stored at ``[j, k]``).
    The batch axis is present only when ``w.batch > 1``.
    """
    A = _draw(w.a_dist, w.dtype, w.seed, TENSOR_A, w.batch * w.M * w.K)
    B = _draw(w.b_dist, w.dtype, w.seed, TENSOR_B, w.batch * w.K * w.N)
    bshape = (w.N, w.K) if w.b_col_major else (w.K, w.N)
    if w.batch > 1:
        return A.reshape(w.batch, w.M, w.K), B.reshape((w.batch,) + bshape)
    return A.reshape(w.M, w.K), B.reshape(bshape)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of ``w`` with some fields replaced (smaller shapes of the same recipe)."""
    d = dict(name=w.name, dtype=w.dtype, M=w.M, N=w.N, K=w.K, seed=w.seed, batch=w.batch, b_col_major=w.b_col_major,
             fixed_k_order=w.fixed_k_order, a_dist=w.a_dist, b_dist=w.b_dist)
    d.update(kw)
    return Workload(**d)


# ---------------------------------------------------------------------- block triangular solve
TENSOR_L = 2
TENSOR_L_DIAG = 3
TENSOR_RHS = 4


@dataclass(frozen=True)
class TrsmWorkload:
    """Synthetic ``L X = B``: ``L`` lower triangular ``[n][n]``, ``B`` ``[n][m]`` (``m`` right-hand sides), fp32.

    ``coupling`` selects the strictly-lower part (``u`` uniform in ``[-1,1)``):

    * ``"dominant"``: ``L_ij = 0.5 * u_ij / i`` -- every row is diagonally dominant (off-diagonal absolute row sum
      below 0.5, diagonal magnitude in ``[1,2)``), so the inverse is bounded by 2 in the infinity norm;
    * ``"sqrt"``: ``L_ij = u_ij / sqrt(n)`` -- the off-diagonal sum of a row is of order one.

    The diagonal is ``+-(1 + v)``, ``v`` uniform in ``[0,1)``, the sign from one more bit.  The strictly upper part is
    filled with ``upper`` (NaN by default: it must never be read).
    """
    name: str
    n: int
    m: int
    tile: int
    seed: int
    coupling: str = "dominant"
    upper: float = float("nan")

    @property
    def flops(self) -> int:
        """Multiply-adds of the substitution counted as two operations: ``n (n+1) m``."""
        return self.n * (self.n + 1) * self.m

    @property
    def algorithmic_bytes(self) -> int:
        """Lower triangle of L and B read once, X written once."""
        return (self.n * (self.n + 1) // 2 + 2 * self.n * self.m) * 4


TRSM_WORKLOADS = {
    "t1": TrsmWorkload("t1", 512, 96, 64, seed=10),
    "t2": TrsmWorkload("t2", 8192, 4096, 256, seed=11),
}


def make_trsm_operands(w: TrsmWorkload):
    """Host arrays ``(L, B)`` (float32) for a triangular-solve workload."""
    n, m = w.n, w.m
    u = uniform_f32(w.seed, TENSOR_L, n * n, -1.0, 1.0).reshape(n, n)
    if w.coupling == "dominant":
        scale = (0.5 / np.maximum(np.arange(n, dtype=np.float64), 1.0)).astype(np.float32)[:, None]
    elif w.coupling == "sqrt":
        scale = np.float32(1.0 / np.sqrt(float(n)))
    else:
        raise ValueError("unknown coupling %r" % (w.coupling,))
    L = (u * scale).astype(np.float32)
    v = uniform_f32(w.seed, TENSOR_L_DIAG, n, 0.0, 1.0)
    sign = np.where((_bits(w.seed, TENSOR_L_DIAG, n, n) >> np.uint64(63)).astype(bool), np.float32(-1.0), np.float32(1.0))
    rows, cols = np.indices((n, n), sparse=True)
    L[rows < cols] = np.float32(w.upper)
    L[np.arange(n), np.arange(n)] = sign * (np.float32(1.0) + v)
    B = uniform_f32(w.seed, TENSOR_RHS, n * m, -1.0, 1.0).reshape(n, m)
    return L, B


# ---------------------------------------------------------------------- FlashAttention-2 recurrence
TENSOR_Q = 5
TENSOR_K = 6
TENSOR_V = 7


@dataclass(frozen=True)
class AttentionWorkload:
    """Synthetic attention problem: ``batch`` independent (Q, K, V) triples, bf16, ``Q`` ``[N][d]``, ``K``/``V`` ``[M][d]``.

    ``Q`` and ``K`` are normal(0, ``qk_std``), ``V`` uniform in ``[-1, 1)``: with unit ``qk_std`` the scaled scores
    ``Q K^T / sqrt(d)`` have unit variance, the regime of a trained attention layer's logits.
    """
    name: str
    batch: int
    N: int
    M: int
    d: int
    seed: int
    qk_std: float = 1.0

    @property
    def flops(self) -> int:
        """Two matrix products per (query, key) pair: ``4 N M d`` per problem."""
        return 4 * self.batch * self.N * self.M * self.d

    @property
    def algorithmic_bytes(self) -> int:
        """Q, K, V read once (bf16), O written once (fp32)."""
        return self.batch * ((self.N + 2 * self.M) * self.d * 2 + self.N * self.d * 4)


ATTENTION_WORKLOADS = {
    "a1": AttentionWorkload("a1", 2, 300, 500, 64, seed=20),
    "a2": AttentionWorkload("a2", 32, 4096, 4096, 128, seed=21),
}


def make_attention_operands(w: AttentionWorkload):
    """Host arrays ``(Q, K, V)`` as bf16 bit patterns (uint16), shapes ``[batch][N][d]`` and ``[batch][M][d]``."""
    Q = f32_to_bf16_bits(normal_f32(w.seed, TENSOR_Q, w.batch * w.N * w.d, w.qk_std)).reshape(w.batch, w.N, w.d)
    K = f32_to_bf16_bits(normal_f32(w.seed, TENSOR_K, w.batch * w.M * w.d, w.qk_std)).reshape(w.batch, w.M, w.d)
    V = f32_to_bf16_bits(uniform_f32(w.seed, TENSOR_V, w.batch * w.M * w.d, -1.0, 1.0)).reshape(w.batch, w.M, w.d)
    return Q, K, V


# ---------------------------------------------------------------------- prefix-sum recurrence
TENSOR_SCAN = 8


@dataclass(frozen=True)
class ScanWorkload:
    """``rows`` independent sequences of ``n`` elements: float32 uniform in ``[-1, 1)`` (running sums that wander around
    zero while ``sum |A|`` grows linearly: the case in which the carried value needs more than fp32), or int32 over the
    whole 32-bit range (running sums that wrap around)."""
    name: str
    rows: int
    n: int
    dtype: str  # "f32" or "i32"
    seed: int

    @property
    def elements(self) -> int:
        return self.rows * self.n

    @property
    def algorithmic_bytes(self) -> int:
        """Each element read once and written once."""
        return 8 * self.rows * self.n


SCAN_WORKLOADS = {
    "p1": ScanWorkload("p1", 3, 10000, "f32", seed=30),
    "p2": ScanWorkload("p2", 1, 1 << 28, "f32", seed=31),
    "p3": ScanWorkload("p3", 4096, 65536, "i32", seed=32),
}


def make_scan_operand(w: ScanWorkload) -> np.ndarray:
    """Host array ``A`` of shape ``[rows][n]``."""
    n = w.rows * w.n
    if w.dtype == "f32":
        return uniform_f32(w.seed, TENSOR_SCAN, n, -1.0, 1.0).reshape(w.rows, w.n)
    if w.dtype == "i32":
        def fn(s, c):
            return (_bits(w.seed, TENSOR_SCAN, s, c) >> np.uint64(32)).astype(np.uint32).view(np.int32)
        return _fill(n, fn, np.int32).reshape(w.rows, w.n)
    raise ValueError("scan workloads are f32 or i32")


# ---------------------------------------------------------------------- Cholesky recurrence
TENSOR_CHOL = 9
TENSOR_CHOL_DIAG = 10


@dataclass(frozen=True)
class CholWorkload:
    """Symmetric positive definite ``A`` of order ``n``: diagonal ``1 + v``, ``v`` uniform in ``[0, 1)``; below the diagonal
    ``coupling = "dominant"``: ``0.5 u_ij / n`` (every row strictly diagonally dominant, so positive definite by
    Gershgorin) or ``"wigner"``: ``0.5 u_ij / sqrt(n)`` (order-one coupling: the off-diagonal part has spectral radius
    about 0.58, eigenvalues of ``A`` stay above 0.4, condition number about 6), ``u`` uniform in ``[-1, 1)``.  Entries
    above the diagonal are NaN: only the lower triangle is an input."""
    name: str
    n: int
    tile: int
    seed: int
    coupling: str = "wigner"

    @property
    def flops(self) -> int:
        """``n^3 / 3`` multiply-adds counted as two operations each, lower-order terms dropped."""
        return self.n ** 3 // 3

    @property
    def algorithmic_bytes(self) -> int:
        """Lower triangle of A read once, lower triangle of L written once."""
        return self.n * (self.n + 1) // 2 * 8


CHOL_WORKLOADS = {
    "h1": CholWorkload("h1", 600, 64, seed=50),
    "h2": CholWorkload("h2", 8192, 256, seed=51),
}


def make_chol_operand(w: CholWorkload) -> np.ndarray:
    """Host array ``A`` ``[n][n]`` float32 with NaN above the diagonal."""
    n = w.n
    scale = 0.5 / n if w.coupling == "dominant" else 0.5 / np.sqrt(n)
    A = (uniform_f32(w.seed, TENSOR_CHOL, n * n, -1.0, 1.0) * np.float32(scale)).reshape(n, n)
    A[np.arange(n), np.arange(n)] = 1.0 + uniform_f32(w.seed, TENSOR_CHOL_DIAG, n, 0.0, 1.0)
    A[np.triu_indices(n, 1)] = np.nan
    return A
