"""The pins must notice plausible mistakes.

Each case plants ONE mistake in a copy of the oracle's source (on the CPU, never in the CUDA
path), builds it to a temporary library and runs the pin file against it in a child process.
The pins have to fail.  Mistakes that would read out of bounds are not planted.
"""
from __future__ import annotations

import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "cq_oracle.c")

MUTATIONS = {
    "row_exponent_swapped": ("pow((double)t[i], alpha)", "pow((double)t[i], 1.0 - alpha)"),
    "col_exponent_swapped": ("pow((double)c[j], 1.0 - alpha)", "pow((double)c[j], alpha)"),
    "qmax_dropped_from_row_factor": ("pow((double)t[i], alpha) / (double)qmax", "pow((double)t[i], alpha)"),
    "round_half_away": ("(int)nearbyintf(u)", "(int)roundf(u)"),
    "truncate_instead_of_round": ("(int)nearbyintf(u)", "(int)truncf(u)"),
    "row_abs_dropped": ("float ax = fabsf(decode16(X[i * ld + j], dtype));\n            if (ax > m) m = ax;\n        }\n        t[i] = m;",
                        "float ax = decode16(X[i * ld + j], dtype);\n            if (ax > m) m = ax;\n        }\n        t[i] = m;"),
    "qmax_is_power_of_two": ("return (1 << (bits - 1)) - 1;", "return (1 << (bits - 1));"),
    "count_only_exact_zero_inputs": ("if (q == 0) zeros += 1;\n            if (codes) codes[i * I + j]", "if (x == 0.0f) zeros += 1;\n            if (codes) codes[i * I + j]"),
    "int4_nibbles_swapped": ("(uint8_t)(lo | (hi << 4))", "(uint8_t)(hi | (lo << 4))"),
    "bf16_encode_truncates": ("if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;", ""),
    "f16_encode_ties_up": ("(rest == 0x1000u && (keep & 1u))", "(rest == 0x1000u)"),
    "f16_decode_exponent_off_by_one": ("e - 25", "e - 24"),
    "weight_scale_uses_qmax_plus_one": ("float d = m / (float)qmax;", "float d = m / (float)(qmax + 1);"),
    "dequant_uses_row_factor_only": ("float xhat = (s == 0.0f) ? 0.0f : (float)q * s;\n            if (q == 0) zeros",
                                     "float xhat = (s == 0.0f) ? 0.0f : (float)q * aa[i];\n            if (q == 0) zeros"),
    "zero_scale_not_guarded": ("if (s == 0.0f) return 0;", ""),
    "col_abs_dropped": ("float ax = fabsf(decode16(X[i * ld + j], dtype));\n            if (ax > m) m = ax;\n        }\n        c[j] = m;",
                        "float ax = decode16(X[i * ld + j], dtype);\n            if (ax > m) m = ax;\n        }\n        c[j] = m;"),
    # Remove Kernel (Figure 1 / Appendix B) and the Table 1 indicators
    "remove_kernel_bound_is_strict": ("int gone = fabsf(u) <= half_bound;", "int gone = fabsf(u) < half_bound;"),
    "remove_kernel_bound_not_halved": ("float half_bound = 0.5f * bound_scale;", "float half_bound = bound_scale;"),
    "remove_kernel_per_token_scale_from_column_maxima": ("float s_pt = t[i] / (float)qmax;\n        for (int64_t j = 0; j < I; ++j) {\n            uint16_t bits16",
                                                          "float s_pt = c[i % I] / (float)qmax;\n        for (int64_t j = 0; j < I; ++j) {\n            uint16_t bits16"),
    "case_two_is_strict": ("if (c[j] >= t[i]) n_case2 += 1;", "if (c[j] > t[i]) n_case2 += 1;"),
    "case_bounds_swapped": ("if (0.5f * s < 0.5f * s_pt) n_smaller += 1;", "if (0.5f * s_pt < 0.5f * s) n_smaller += 1;"),
    # alpha = 0 evaluated through the general branch: s = fl32(fl32(1/qmax) * c) instead of fl32(c/qmax)
    "alpha_zero_not_special_cased": [("else if (alpha == 0.0) a[i] = 1.0f;", ""),
                                     ("else if (alpha == 0.0) b[j] = c[j] / (float)qmax;", "")],
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(name, tmp_path):
    edits = MUTATIONS[name]
    if isinstance(edits, tuple):
        edits = [edits]
    mutated = open(SRC).read()
    for old, new in edits:
        assert mutated.count(old) >= 1, f"mutation target not found: {name}"
        mutated = mutated.replace(old, new, 1)
    src = tmp_path / "cq_oracle_mut.c"
    lib = tmp_path / "libcq_oracle_mut.so"
    src.write_text(mutated)
    subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                    "-o", str(lib), str(src), "-lm"], check=True)
    env = dict(os.environ, CQ_ORACLE_LIB=str(lib))
    # the exhaustive, 50-digit and torch-importing pins are left out here only to keep this file quick
    proc = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                           "-k", "not all_2x2 and not random_2x3 and not decimal and not torch",
                           os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                          cwd=ROOT, env=env, capture_output=True, text=True)
    assert proc.returncode != 0, f"no pin noticed the planted mistake {name!r}"
    assert "failed" in proc.stdout or "error" in proc.stdout.lower()
