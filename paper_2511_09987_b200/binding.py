"""ctypes binding of ``libcyc.so`` (see ``include/cyc.h``): argument marshalling only.

The functions named ``cyc_*`` take the same arguments as the C entry points
(integers and raw device/host addresses).  :func:`recurrence_matmul`,
:func:`recurrence_matmul_batched` and :func:`recurrence_matmul_host` accept torch
tensors, allocate the result with torch and pass the current torch stream; every
step of the computation runs in the library's kernels.  There is no CPU fallback:
if the library is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libcyc.so")

CYC_F32, CYC_BF16_F32, CYC_I8_I32, CYC_I32 = 0, 1, 2, 3
CYC_FLAG_FIXED_K_ORDER, CYC_FLAG_B_COL_MAJOR = 1, 2
CYC_OK, CYC_ERR_INVALID_ARG, CYC_ERR_UNSUPPORTED, CYC_ERR_CUDA, CYC_ERR_TIMEOUT = 0, 1, 2, 3, 4
DTYPE_CODES = {"f32": CYC_F32, "bf16": CYC_BF16_F32, "i8": CYC_I8_I32}

# every symbol include/cyc.h declares: name -> (restype, argtypes)
_i64, _int, _u32, _ptr = ctypes.c_int64, ctypes.c_int, ctypes.c_uint, ctypes.c_void_p
SYMBOLS = {
    "cyc_recurrence_matmul": (_int, [_i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _ptr, _u32]),
    "cyc_recurrence_matmul_batched": (_int, [_i64, _i64, _i64, _i64, _int, _ptr, _i64, _ptr, _i64, _ptr, _i64, _ptr, _u32]),
    "cyc_recurrence_matmul_host": (_int, [_i64, _i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _ptr, _u32]),
    "cyc_recurrence_matmul_splitk_static": (_int, [_i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _ptr, _u32]),
    "cyc_pool_reserved_bytes": (_int, [ctypes.POINTER(ctypes.c_int64)]),
    "cyc_block_trsm": (_int, [_i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _ptr, _u32]),
    "cyc_flash_attention": (_int, [_i64, _i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _ptr, _ptr, _u32]),
    "cyc_prefix_sum": (_int, [_i64, _i64, _int, _ptr, _i64, _ptr, _i64, _ptr, _u32]),
    "cyc_cholesky": (_int, [_i64, _i64, _int, _ptr, _ptr, _ptr, _u32]),
    "cyc_selftest_bounded_wait": (_int, [_ptr, _i64]),
    "cyc_last_device_status": (_int, [_ptr, ctypes.POINTER(ctypes.c_int)]),
    "cyc_kernel_for": (ctypes.c_char_p, [_i64, _i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _u32]),
    "cyc_schedule_for": (ctypes.c_char_p, [_i64, _i64, _i64, _i64, _int, _ptr, _ptr, _ptr, _u32]),
    "cyc_launch_count": (_i64, []),
    "cyc_last_cuda_error": (ctypes.c_char_p, []),
    "cyc_status_string": (ctypes.c_char_p, [_int]),
    "cyc_version": (_int, []),
}


class CycError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        name = _lib.cyc_status_string(status).decode()
        super().__init__("cyc: %s (status %d)%s" % (name, status, (": " + detail) if detail else ""))


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2511_09987_b200.build`" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)  # AttributeError if the library does not export it
        fn.restype, fn.argtypes = res, args
    return lib


_lib = _load()

cyc_recurrence_matmul = _lib.cyc_recurrence_matmul
cyc_recurrence_matmul_batched = _lib.cyc_recurrence_matmul_batched
cyc_recurrence_matmul_host = _lib.cyc_recurrence_matmul_host
cyc_recurrence_matmul_splitk_static = _lib.cyc_recurrence_matmul_splitk_static
cyc_pool_reserved_bytes = _lib.cyc_pool_reserved_bytes
cyc_block_trsm = _lib.cyc_block_trsm
cyc_flash_attention = _lib.cyc_flash_attention
cyc_prefix_sum = _lib.cyc_prefix_sum
cyc_cholesky = _lib.cyc_cholesky
cyc_selftest_bounded_wait = _lib.cyc_selftest_bounded_wait
cyc_last_device_status = _lib.cyc_last_device_status
CYC_STATIC_WORKSPACE_BYTES = 8 << 20
cyc_kernel_for = _lib.cyc_kernel_for
cyc_schedule_for = _lib.cyc_schedule_for
cyc_launch_count = _lib.cyc_launch_count
cyc_last_cuda_error = _lib.cyc_last_cuda_error
cyc_status_string = _lib.cyc_status_string
cyc_version = _lib.cyc_version


def check(status: int) -> None:
    if status != CYC_OK:
        raise CycError(status, cyc_last_cuda_error().decode() if status in (CYC_ERR_CUDA, CYC_ERR_UNSUPPORTED) else "")


def _flags(b_col_major: bool, fixed_k_order: bool) -> int:
    return (CYC_FLAG_B_COL_MAJOR if b_col_major else 0) | (CYC_FLAG_FIXED_K_ORDER if fixed_k_order else 0)


def _torch_dtype_code(t) -> int:
    import torch
    return {torch.float32: CYC_F32, torch.bfloat16: CYC_BF16_F32, torch.int8: CYC_I8_I32}[t.dtype]


def _stream(t=None) -> int:
    """The current torch stream of the device the operands live on (which must be the current device: the library
    launches on the current device)."""
    import torch
    if t is not None and t.device.index != torch.cuda.current_device():
        raise ValueError("operands live on %s but the current device is cuda:%d" % (t.device, torch.cuda.current_device()))
    return torch.cuda.current_stream().cuda_stream


def _check_out(name, T, shape, dtype, like):
    """A caller-supplied result tensor goes to the kernels as a raw address: refuse anything but a contiguous CUDA
    tensor of the exact shape and dtype on the operands' device."""
    if not (T.is_cuda and T.device == like.device and T.is_contiguous() and tuple(T.shape) == tuple(shape) and T.dtype == dtype):
        raise ValueError("%s must be a contiguous %s CUDA tensor of shape %s on %s" % (name, dtype, tuple(shape), like.device))


def recurrence_matmul(A, B, C=None, *, b_col_major: bool = False, fixed_k_order: bool = False):
    """``C[M,N] = sum_k A[M,K] B[K,N]`` for CUDA tensors (B is ``[N,K]`` when ``b_col_major``)."""
    import torch
    if not (A.is_cuda and B.is_cuda and A.is_contiguous() and B.is_contiguous() and A.dim() == 2 and B.dim() == 2):
        raise ValueError("A and B must be contiguous CUDA matrices")
    code = _torch_dtype_code(A)
    if B.dtype != A.dtype:
        raise ValueError("A and B must have the same dtype")
    M, K = A.shape
    N = B.shape[0] if b_col_major else B.shape[1]
    if (B.shape[1] if b_col_major else B.shape[0]) != K:
        raise ValueError("inner dimensions differ")
    out_dtype = torch.int32 if code == CYC_I8_I32 else torch.float32
    if B.device != A.device:
        raise ValueError("A and B must live on the same device")
    if C is None:
        C = torch.empty((M, N), dtype=out_dtype, device=A.device)
    else:
        _check_out("C", C, (M, N), out_dtype, A)
    check(cyc_recurrence_matmul(M, N, K, code, A.data_ptr(), B.data_ptr(), C.data_ptr(), _stream(A),
                                _flags(b_col_major, fixed_k_order)))
    return C


def recurrence_matmul_batched(A, B, C=None, *, b_col_major: bool = False, fixed_k_order: bool = False):
    """Batched form for contiguous ``A[batch,M,K]``, ``B[batch,K,N]`` (or ``[batch,N,K]``)."""
    import torch
    if not (A.is_cuda and B.is_cuda and A.is_contiguous() and B.is_contiguous() and A.dim() == 3 and B.dim() == 3):
        raise ValueError("A and B must be contiguous CUDA tensors of rank 3")
    code = _torch_dtype_code(A)
    batch, M, K = A.shape
    N = B.shape[1] if b_col_major else B.shape[2]
    if B.shape[0] != batch or (B.shape[2] if b_col_major else B.shape[1]) != K or B.dtype != A.dtype:
        raise ValueError("operand shapes or dtypes differ")
    out_dtype = torch.int32 if code == CYC_I8_I32 else torch.float32
    if B.device != A.device:
        raise ValueError("A and B must live on the same device")
    if C is None:
        C = torch.empty((batch, M, N), dtype=out_dtype, device=A.device)
    else:
        _check_out("C", C, (batch, M, N), out_dtype, A)
    check(cyc_recurrence_matmul_batched(batch, M, N, K, code, A.data_ptr(), 0, B.data_ptr(), 0, C.data_ptr(), 0, _stream(A),
                                        _flags(b_col_major, fixed_k_order)))
    return C


def recurrence_matmul_host(A, B, C, *, b_col_major: bool = False, fixed_k_order: bool = False):
    """Host tensors in, host tensor out (copies inside the call); ``A`` is ``[M,K]`` or ``[batch,M,K]``."""
    if A.is_cuda or B.is_cuda or C.is_cuda:
        raise ValueError("host tensors expected")
    code = _torch_dtype_code(A)
    if A.dim() == 2:
        batch, (M, K) = 1, A.shape
        N = B.shape[0] if b_col_major else B.shape[1]
    else:
        batch, M, K = A.shape
        N = B.shape[1] if b_col_major else B.shape[2]
    if C.numel() != batch * M * N or not (A.is_contiguous() and B.is_contiguous() and C.is_contiguous()):
        raise ValueError("bad result shape or non-contiguous tensors")
    check(cyc_recurrence_matmul_host(batch, M, N, K, code, A.data_ptr(), B.data_ptr(), C.data_ptr(), _stream(),
                                     _flags(b_col_major, fixed_k_order)))
    return C


def recurrence_matmul_splitk_static(A, B, C=None, *, b_col_major: bool = False):
    """Split-K evaluation through the library's fixed workspace: the call itself allocates nothing.

    For hosts that must not allocate device memory at call time; pass ``C`` to keep torch from allocating
    the result as well.  bf16 or int8 CUDA matrices with M, N > 128; see ``include/cyc.h`` for the size limit.
    Calls share one workspace: keep them ordered on a stream."""
    import torch
    if not (A.is_cuda and B.is_cuda and A.is_contiguous() and B.is_contiguous() and A.dim() == 2 and B.dim() == 2):
        raise ValueError("A and B must be contiguous CUDA matrices")
    code = _torch_dtype_code(A)
    M, K = A.shape
    N = B.shape[0] if b_col_major else B.shape[1]
    if (B.shape[1] if b_col_major else B.shape[0]) != K or B.dtype != A.dtype:
        raise ValueError("operand shapes or dtypes differ")
    out_dtype = torch.int32 if code == CYC_I8_I32 else torch.float32
    if B.device != A.device:
        raise ValueError("A and B must live on the same device")
    if C is None:
        C = torch.empty((M, N), dtype=out_dtype, device=A.device)
    else:
        _check_out("C", C, (M, N), out_dtype, A)
    check(cyc_recurrence_matmul_splitk_static(M, N, K, code, A.data_ptr(), B.data_ptr(), C.data_ptr(), _stream(A),
                                              _flags(b_col_major, False)))
    return C


def block_trsm(L, B, X=None, *, tile: int = 0, fixed_k_order: bool = False):
    """Solve ``L X = B`` for contiguous fp32 CUDA tensors ``L[n,n]`` (lower triangle read) and ``B[n,m]``.

    ``X`` defaults to a new tensor; pass ``X=B`` to solve in place."""
    import torch
    if not (L.is_cuda and B.is_cuda and L.is_contiguous() and B.is_contiguous() and L.dim() == 2 and B.dim() == 2):
        raise ValueError("L and B must be contiguous CUDA matrices")
    n, m = B.shape
    if L.shape[0] != n or L.shape[1] != n or L.dtype != B.dtype:
        raise ValueError("L must be [n,n] and B [n,m] of one dtype")
    if X is None:
        X = torch.empty_like(B)
    elif not (X.is_cuda and X.device == B.device and X.is_contiguous() and X.shape == B.shape and X.dtype == B.dtype):
        raise ValueError("X must be a contiguous CUDA tensor shaped like B")
    if L.device != B.device:
        raise ValueError("L and B must live on the same device")
    check(cyc_block_trsm(n, m, tile, _torch_dtype_code(L), L.data_ptr(), B.data_ptr(), X.data_ptr(), _stream(L),
                         _flags(False, fixed_k_order)))
    return X


def flash_attention(Q, K, V, O=None):
    """``softmax(Q K^T / sqrt(d)) V`` by the FlashAttention-2 recurrence for contiguous bf16 CUDA tensors
    ``Q[batch,N,d]``, ``K[batch,M,d]``, ``V[batch,M,d]`` (or rank 2 for one problem); fp32 result shaped like ``Q``."""
    import torch
    if Q.dim() == 2:
        Q, K, V = Q.unsqueeze(0), K.unsqueeze(0), V.unsqueeze(0)
        squeeze = True
    else:
        squeeze = False
    if not all(t.is_cuda and t.is_contiguous() and t.dim() == 3 for t in (Q, K, V)):
        raise ValueError("Q, K, V must be contiguous CUDA tensors of rank 2 or 3")
    batch, N, d = Q.shape
    M = K.shape[1]
    if K.shape != (batch, M, d) or V.shape != (batch, M, d) or K.dtype != Q.dtype or V.dtype != Q.dtype:
        raise ValueError("operand shapes or dtypes differ")
    if K.device != Q.device or V.device != Q.device:
        raise ValueError("Q, K and V must live on the same device")
    if O is None:
        O = torch.empty((batch, N, d), dtype=torch.float32, device=Q.device)
    else:
        if O.dim() == 2 and squeeze:
            O = O.unsqueeze(0)
        _check_out("O", O, (batch, N, d), torch.float32, Q)
    check(cyc_flash_attention(batch, N, M, d, _torch_dtype_code(Q), Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(),
                              _stream(Q), 0))
    return O[0] if squeeze else O


def prefix_sum(A, P=None):
    """Inclusive prefix sums ``P_i = P_{i-1} + A_i`` along the last dimension of a CUDA tensor ``A`` of rank 1 or 2
    (float32 or int32; rows of a rank-2 tensor are independent sequences and may be strided).  ``P`` may be ``A``."""
    import torch
    if not A.is_cuda or A.dim() not in (1, 2) or A.stride(-1) != 1:
        raise ValueError("A must be a CUDA tensor of rank 1 or 2 with a contiguous last dimension")
    codes = {torch.float32: CYC_F32, torch.int32: CYC_I32}
    if A.dtype not in codes:
        raise ValueError("float32 or int32 only")
    if P is None:
        P = torch.empty(A.shape, dtype=A.dtype, device=A.device)
    if P.shape != A.shape or P.dtype != A.dtype or not P.is_cuda or P.device != A.device or P.stride(-1) != 1:
        raise ValueError("P must match A")
    rows, n = (1, A.shape[0]) if A.dim() == 1 else A.shape
    if rows * n == 0:
        return P
    sA = A.stride(0) if A.dim() == 2 and rows > 1 else n
    sP = P.stride(0) if P.dim() == 2 and rows > 1 else n
    check(cyc_prefix_sum(rows, n, codes[A.dtype], A.data_ptr(), sA, P.data_ptr(), sP, _stream(A), 0))
    return P


def cholesky(A, L=None, *, tile: int = 0, fixed_k_order: bool = False):
    """Lower Cholesky factor of the symmetric positive definite float32 CUDA matrix ``A[n,n]`` (only its lower triangle is
    read) by the tiled recurrence; ``L`` may be ``A`` (in place)."""
    import torch
    if not (A.is_cuda and A.is_contiguous() and A.dim() == 2 and A.shape[0] == A.shape[1] and A.dtype == torch.float32):
        raise ValueError("A must be a contiguous square float32 CUDA tensor")
    if L is None:
        L = torch.empty_like(A)
    if L.shape != A.shape or L.dtype != A.dtype or not L.is_cuda or L.device != A.device or not L.is_contiguous():
        raise ValueError("L must match A")
    check(cyc_cholesky(A.shape[0], tile, CYC_F32, A.data_ptr(), L.data_ptr(), _stream(A), _flags(False, fixed_k_order)))
    return L


def last_device_status() -> int:
    out = ctypes.c_int(0)
    check(cyc_last_device_status(_stream(), ctypes.byref(out)))
    return out.value


def kernel_for(batch, M, N, K, dtype, a_ptr=256, b_ptr=1 << 40, c_ptr=1 << 41, *, b_col_major=False, fixed_k_order=False):
    r = cyc_kernel_for(batch, M, N, K, DTYPE_CODES.get(dtype, dtype), a_ptr, b_ptr, c_ptr, _flags(b_col_major, fixed_k_order))
    return r.decode() if r else None


def schedule_for(batch, M, N, K, dtype, a_ptr=256, b_ptr=1 << 40, c_ptr=1 << 41, *, b_col_major=False, fixed_k_order=False):
    r = cyc_schedule_for(batch, M, N, K, DTYPE_CODES.get(dtype, dtype), a_ptr, b_ptr, c_ptr, _flags(b_col_major, fixed_k_order))
    return r.decode() if r else None
