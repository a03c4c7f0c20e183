"""The pins have teeth: each planted mistake in a copy of the oracle's C source (compiled into a
temporary library, on the CPU) is caught by at least one pin of test_oracle_pins."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

HERE = os.path.dirname(os.path.abspath(oracle.__file__))

# (name, file, original text, planted text)
MUTANTS = [
    ("collapsed_walks_k_downwards", "cyc_oracle_walkers.inc",
     "for (int64_t k = 0; k < K; ++k) {\n            T w = A[i * K + k];",
     "for (int64_t k = K - 1; k >= 0; --k) {\n            T w = A[i * K + k];"),
    ("literal_partial_sum_starts_at_one", "cyc_oracle_walkers.inc", "cin = (T)0;\n                    if (cnt) cnt[ST_ZERO_C]++;\n                } else {\n                    if (!fromW[me].full)",
     "cin = (T)1;\n                    if (cnt) cnt[ST_ZERO_C]++;\n                } else {\n                    if (!fromW[me].full)"),
    ("subtracts_the_product", "cyc_oracle.c", "return cin + p;", "return cin - p;"),
    ("fused_and_separate_swapped", "cyc_oracle.c", "if (fma) return fmaf(w, b, cin);", "if (!fma) return fmaf(w, b, cin);"),
    ("weights_loaded_mirrored_in_k", "cyc_oracle_walkers.inc", "W[i * K + k] = A[i * K + k];\n            if (counts) counts[cell_type(i, k, M, K) * ST_COUNT + ST_LOAD_W]++;\n        }\n    for (int64_t j = 0; j < N && !rc; ++j) {",
     "W[i * K + k] = A[i * K + (K - 1 - k)];\n            if (counts) counts[cell_type(i, k, M, K) * ST_COUNT + ST_LOAD_W]++;\n        }\n    for (int64_t j = 0; j < N && !rc; ++j) {"),
    ("bf16_widened_with_wrong_shift", "cyc_oracle.c", "uint32_t u = ((uint32_t)h) << 16;", "uint32_t u = ((uint32_t)h) << 15;"),
    ("wavefront_ignores_the_k_skew", "cyc_oracle_walkers.inc", "int64_t j = t - i - k; /* the time step this cell is at: t = i + j + k */",
     "int64_t j = t - i; /* planted */"),
    ("last_row_still_sends_b_south", "cyc_oracle_walkers.inc", "if (i + 1 < M) {\n                    size_t to = (size_t)((i + 1) * K + k);\n                    if (fromN[to].full) { rc = ORC_CHANNEL; break; }",
     "if (1) {\n                    size_t to = (size_t)(((i + 1) % M) * K + k);\n                    if (fromN[to].full) { rc = ORC_CHANNEL; break; }"),
    ("b_read_transposed_when_column_major", "cyc_oracle.c", "int64_t brs = b_col_major ? 1 : N, bcs = b_col_major ? K : 1;\n    if (dtype == CYC_ORACLE_I8_I32) {\n        *Aw",
     "int64_t brs = N, bcs = 1;\n    if (dtype == CYC_ORACLE_I8_I32) {\n        *Aw"),
    ("points_start_from_one", "cyc_oracle.c", "float c = 0.0f;\n            for (int64_t k = 0; k < K; ++k) c = mac_f(c, ((const float *)A)",
     "float c = 1.0f;\n            for (int64_t k = 0; k < K; ++k) c = mac_f(c, ((const float *)A)"),
]


def _pins():
    """A representative subset of the pins, as zero-argument callables."""
    out = []
    for dtype in ("f32", "bf16", "i8"):
        for mode in pins.ALL_MODES:
            out.append(lambda d=dtype, m=mode: pins.test_identity_and_permutation(d, m))
            out.append(lambda d=dtype, m=mode: pins.test_all_ones(d, m, (5, 3, 64)))
            out.append(lambda d=dtype, m=mode: pins.test_brute_force_tiny_exact(d, m))
    for case in pins._cases():
        for mode in pins.ALL_MODES:
            out.append(lambda c=case, m=mode: pins.test_ieee_order_cases(c, m))
    out.append(pins.test_bf16_widening_values)
    for mode in ("literal", "wavefront"):
        out.append(lambda m=mode: pins.test_nine_cell_programs(m, (3, 3)))
    out.append(lambda: pins.test_modes_agree("f32", False, True))
    return out


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(mutant, tmp_path, monkeypatch):
    name, fname, old, new = mutant
    for f in ("cyc_oracle.c", "cyc_oracle_walkers.inc"):
        text = open(os.path.join(HERE, f)).read()
        if f == fname:
            assert text.count(old) >= 1, "mutation site not found: the oracle source changed, update this test"
            text = text.replace(old, new, 1)
        (tmp_path / f).write_text(text)
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", *oracle.CFLAGS, "-o", lib_path, str(tmp_path / "cyc_oracle.c"), "-lm"])
    monkeypatch.setattr(oracle, "_lib", ctypes.CDLL(lib_path))
    caught = 0
    for pin in _pins():
        try:
            pin()
        except (AssertionError, RuntimeError, OverflowError, ValueError):
            caught += 1
    assert caught > 0, "no pin noticed the planted mistake %r" % name


def test_unmodified_oracle_passes_the_same_pins():
    for pin in _pins():
        pin()
