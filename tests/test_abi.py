"""The C ABI without a GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before any CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2511_09987_b200 import build
    build.build()
    from paper_2511_09987_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cyc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cyc_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(binding):
    names = declared_symbols()
    assert "cyc_recurrence_matmul" in names and "cyc_recurrence_matmul_batched" in names
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.SYMBOLS) == names


def test_status_strings_and_version(binding):
    assert binding.cyc_version() >= 100
    assert binding.cyc_status_string(0) == b"ok"
    assert binding.cyc_status_string(4) == b"device wait timed out"
    assert binding.cyc_launch_count() >= 0


def test_invalid_arguments_rejected_on_host(binding):
    b = binding
    A, B, C = 1 << 20, 1 << 30, 1 << 40   # never dereferenced: validation comes first
    f = b.cyc_recurrence_matmul
    assert f(0, 4, 4, 0, A, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, -1, 4, 0, A, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, 4, 0, 0, A, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, 4, 4, 7, A, B, C, None, 0) == b.CYC_ERR_INVALID_ARG          # unknown dtype
    assert f(4, 4, 4, 0, A, B, C, None, 8) == b.CYC_ERR_INVALID_ARG          # unknown flag
    assert f(4, 4, 4, 0, None, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, 4, 4, 0, A, None, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, 4, 4, 0, A, B, None, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(4, 4, 4, 0, A + 2, B, C, None, 0) == b.CYC_ERR_INVALID_ARG      # fp32 operand not 4-byte aligned
    assert f(4, 4, 4, 0, A, B, A + 16, None, 0) == b.CYC_ERR_INVALID_ARG     # C overlaps A
    assert f(4, 4, 131072, 2, A, B, C, None, 0) == b.CYC_ERR_UNSUPPORTED     # int32 could overflow
    g = b.cyc_recurrence_matmul_batched
    assert g(0, 4, 4, 4, 0, A, 0, B, 0, C, 0, None, 0) == b.CYC_ERR_INVALID_ARG
    assert g(2, 4, 4, 4, 0, A, 15, B, 0, C, 0, None, 0) == b.CYC_ERR_INVALID_ARG   # stride smaller than a matrix
    assert g(2, 4, 4, 4, 0, A, 0, B, 0, C, -1, None, 0) == b.CYC_ERR_INVALID_ARG
    h = b.cyc_recurrence_matmul_host
    assert h(1, 4, 4, 4, 0, None, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
    assert h(1, 4, 4, 4, 9, A, B, C, None, 0) == b.CYC_ERR_INVALID_ARG


def test_block_trsm_arguments_rejected_on_host(binding):
    b = binding
    L, B, X = 1 << 20, 1 << 30, 1 << 40   # never dereferenced: validation comes first
    t = b.cyc_block_trsm
    assert t(0, 4, 0, 0, L, B, X, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 0, 0, 0, L, B, X, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 4, 257, 0, L, B, X, None, 0) == b.CYC_ERR_INVALID_ARG         # tile edge above 256
    assert t(4, 4, -1, 0, L, B, X, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 4, 0, 5, L, B, X, None, 0) == b.CYC_ERR_INVALID_ARG           # unknown dtype
    assert t(4, 4, 0, 1, L, B, X, None, 0) == b.CYC_ERR_UNSUPPORTED           # bf16: the solve is fp32 only
    assert t(4, 4, 0, 2, L, B, X, None, 0) == b.CYC_ERR_UNSUPPORTED
    assert t(4, 4, 0, 0, L, B, X, None, 2) == b.CYC_ERR_INVALID_ARG           # no column-major flag here
    assert t(4, 4, 0, 0, None, B, X, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 4, 0, 0, L, None, X, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 4, 0, 0, L, B, None, None, 0) == b.CYC_ERR_INVALID_ARG
    assert t(4, 4, 0, 0, L, B + 2, X, None, 0) == b.CYC_ERR_INVALID_ARG       # not 4-byte aligned
    assert t(4, 4, 0, 0, L, B, L + 32, None, 0) == b.CYC_ERR_INVALID_ARG      # X over L
    assert t(4, 4, 0, 0, L, B, B + 16, None, 0) == b.CYC_ERR_INVALID_ARG      # X over B, not in place
    assert t(1 << 31, 4, 0, 0, L, B, X, None, 0) == b.CYC_ERR_UNSUPPORTED


def test_flash_attention_arguments_rejected_on_host(binding):
    b = binding
    Q, K, V, O = 1 << 20, 1 << 30, 1 << 34, 1 << 40   # never dereferenced: validation comes first
    f = b.cyc_flash_attention
    assert f(0, 8, 8, 64, 1, Q, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 0, 8, 64, 1, Q, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, -3, 64, 1, Q, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, 8, 64, 9, Q, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG          # unknown dtype
    assert f(1, 8, 8, 64, 1, Q, K, V, O, None, 1) == b.CYC_ERR_INVALID_ARG          # no flag applies
    assert f(1, 8, 8, 64, 1, None, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, 8, 64, 1, Q, K, V, None, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, 8, 64, 1, Q + 1, K, V, O, None, 0) == b.CYC_ERR_INVALID_ARG      # bf16 operand not 2-byte aligned
    assert f(1, 8, 8, 64, 1, Q, K, V, Q + 64, None, 0) == b.CYC_ERR_INVALID_ARG     # O over Q
    assert f(1, 8, 8, 64, 0, Q, K, V, O, None, 0) == b.CYC_ERR_UNSUPPORTED          # fp32 inputs
    assert f(1, 8, 8, 96, 1, Q, K, V, O, None, 0) == b.CYC_ERR_UNSUPPORTED          # head dimension
    assert f(1, 8, 8, 64, 1, Q + 2, K, V, O, None, 0) == b.CYC_ERR_UNSUPPORTED      # not 16-byte aligned


def test_prefix_sum_arguments_rejected_on_host(binding):
    b = binding
    A, P = 1 << 20, 1 << 30   # never dereferenced: validation comes first
    f = b.cyc_prefix_sum
    assert f(0, 8, 0, A, 0, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 0, 0, A, 0, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, 9, A, 0, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG                # unknown dtype
    assert f(1, 8, 0, A, 0, P, 0, None, 1) == b.CYC_ERR_INVALID_ARG                # no flag applies
    assert f(1, 8, 0, None, 0, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(1, 8, 0, A, 0, None, 0, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(2, 8, 0, A, 7, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG                # stride shorter than a sequence
    assert f(1, 8, 0, A + 2, 0, P, 0, None, 0) == b.CYC_ERR_INVALID_ARG            # not 4-byte aligned
    assert f(1, 8, 0, A, 0, A + 16, 0, None, 0) == b.CYC_ERR_INVALID_ARG           # P over A, other than in place
    assert f(2, 8, 0, A, 8, A, 16, None, 0) == b.CYC_ERR_INVALID_ARG               # same base, different strides
    assert f(1, 8, 1, A, 0, P, 0, None, 0) == b.CYC_ERR_UNSUPPORTED                # bf16
    assert f(1, 8, 2, A, 0, P, 0, None, 0) == b.CYC_ERR_UNSUPPORTED                # int8
    assert f(1, (1 << 40) + 1, 3, A, 0, P, 0, None, 0) == b.CYC_ERR_UNSUPPORTED    # sequence too long
    assert f(1 << 22, 1 << 24, 3, A, 0, 1 << 50, 0, None, 0) == b.CYC_ERR_UNSUPPORTED  # 2^32 tiles


def test_cholesky_arguments_rejected_on_host(binding):
    b = binding
    A, L = 1 << 20, 1 << 40   # never dereferenced: validation comes first
    f = b.cyc_cholesky
    assert f(0, 0, 0, A, L, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(8, -1, 0, A, L, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(8, 257, 0, A, L, None, 0) == b.CYC_ERR_INVALID_ARG                  # tile edge above 256
    assert f(8, 0, 9, A, L, None, 0) == b.CYC_ERR_INVALID_ARG                    # unknown dtype
    assert f(8, 0, 0, A, L, None, 2) == b.CYC_ERR_INVALID_ARG                    # only the fixed-k-order flag applies
    assert f(8, 0, 0, None, L, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(8, 0, 0, A, None, None, 0) == b.CYC_ERR_INVALID_ARG
    assert f(8, 0, 0, A + 2, L, None, 0) == b.CYC_ERR_INVALID_ARG                # not 4-byte aligned
    assert f(8, 0, 0, A, A + 64, None, 0) == b.CYC_ERR_INVALID_ARG               # overlap other than in place
    assert f(8, 0, 1, A, L, None, 0) == b.CYC_ERR_UNSUPPORTED                    # bf16
    assert f(1 << 31, 0, 0, A, 1 << 62, None, 0) == b.CYC_ERR_UNSUPPORTED


def test_kernel_selection(binding):
    k = binding.kernel_for
    assert k(1, 64, 64, 64, "f32", fixed_k_order=True) == "simt"
    assert k(1, 8192, 8192, 8192, "bf16") == "tcgen05_pair_tall"
    assert k(1, 4096, 4096, 4096, "i8", b_col_major=True) == "tcgen05_pair"    # 32 k-blocks: 256x256 tiles
    assert k(1, 4096, 4096, 16384, "i8", b_col_major=True) == "tcgen05_pair_tall"
    assert k(1024, 256, 256, 256, "bf16") == "tcgen05_pair"
    assert k(1, 4096, 4096, 64, "bf16") == "tcgen05_pair"        # k loop too short for the tall tiles
    assert k(1, 128, 4096, 4096, "bf16") == "tcgen05"            # one row block: a single CTA per tile
    assert k(1, 256, 256, 8192, "bf16") == "tcgen05_pair_splitk" # one tile, 128 k-blocks
    assert k(1, 256, 256, 8192, "bf16", fixed_k_order=True) == "tcgen05_pair"
    assert k(1, 256, 256, 512, "bf16") == "tcgen05_pair"         # k loop too short to cut
    assert k(1, 65536, 256, 256, "f32") == "tcgen05_3xtf32_ws"   # small B under a long A: B stays in tensor memory
    assert k(1, 65536, 256, 256, "f32", b_col_major=True) == "tcgen05_3xtf32_ws"
    assert k(1, 65536, 256, 512, "f32") == "tcgen05_3xtf32"      # B too large to stay
    assert k(1, 4096, 256, 256, "f32") == "tcgen05_3xtf32"       # too few rows to pay for the prologue
    assert k(4, 65536, 256, 256, "f32") == "tcgen05_3xtf32"
    assert k(1, 65536, 64, 256, "f32") == "tcgen05_3xtf32_ws"    # fewer columns than a CTA pair's tile: still the tensor cores
    assert k(1, 65536, 8, 256, "f32") == "tcgen05_3xtf32_ws"
    assert k(1, 65536, 62, 256, "f32") == "simt"                 # row pitch of B and C not a multiple of 16 bytes
    assert k(1, 65536, 128, 512, "f32") == "simt"
    assert k(1, 65536, 256, 256, "f32", fixed_k_order=True) == "simt"
    assert k(1, 128, 256, 256, "f32") == "simt"
    assert k(1, 65, 127, 33, "bf16") == "simt"               # pitches not multiples of 16 bytes
    assert k(1, 64, 64, 64, "bf16", a_ptr=258) == "simt"     # base not 16-byte aligned
    assert k(1, 64, 64, 64, "bf16", a_ptr=257) is None       # not even element aligned
    assert k(1, 0, 64, 64, "bf16") is None


def test_static_workspace_entry_point_refuses_on_the_host(binding):
    """Requests the fixed workspace cannot serve are turned down by host-side checks, before any CUDA call."""
    b = binding
    A, B, C = 1 << 20, 1 << 30, 1 << 40       # never dereferenced: the checks come before any launch
    f = b.cyc_recurrence_matmul_splitk_static
    big = 2048                                 # 2 * 2048 * 2048 * 4 bytes = 32 MiB > 8 MiB
    assert 2 * big * big * 4 > b.CYC_STATIC_WORKSPACE_BYTES
    assert f(big, big, 8192, b.CYC_BF16_F32, A, B, C, None, 0) == b.CYC_ERR_UNSUPPORTED
    assert b"fixed workspace" in b.cyc_last_cuda_error()
    assert f(256, 256, 512, b.CYC_BF16_F32, A, B, C, None, 0) == b.CYC_ERR_UNSUPPORTED       # k loop too short to cut
    assert f(256, 256, 8192, b.CYC_F32, A, B, C, None, 0) == b.CYC_ERR_UNSUPPORTED           # fp32 has no split-K path
    assert f(256, 256, 8192, b.CYC_BF16_F32, A, B, C, None, b.CYC_FLAG_FIXED_K_ORDER) == b.CYC_ERR_INVALID_ARG
    assert f(256, 256, 8192, b.CYC_BF16_F32, None, B, C, None, 0) == b.CYC_ERR_INVALID_ARG
