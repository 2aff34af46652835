"""The C-ABI library: it loads, exports every symbol cq.h declares, and rejects bad arguments
before touching the GPU (so these run on a machine without one)."""
from __future__ import annotations

import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2410_07505_b200 import build, cq
    build.build()
    return cq.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cq_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_symbols()
    for must in ("cq_absmax_rows", "cq_absmax_cols", "cq_quantize_act", "cq_dequantize", "cq_kernel_count",
                 "cq_quantize_weight_per_channel"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    from paper_2410_07505_b200 import cq
    names = declared_symbols()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), f"{name} declared in cq.h but not exported"
    assert set(cq.EXPORTS) == set(names)


def test_status_strings(lib):
    from paper_2410_07505_b200 import cq
    assert cq.version() >= 100
    seen = {cq.status_string(s) for s in range(10)}
    assert len(seen) == 10 and cq.status_string(0) == "ok"
    assert cq.status_string(99) == "unknown status"


def test_workspace_size_grows_with_the_matrix(lib):
    from paper_2410_07505_b200 import cq
    small, big = cq.workspace_bytes(128, 768), cq.workspace_bytes(4096, 28672)
    assert 0 < small < big < 64 * 2 ** 20
    assert cq.workspace_bytes(0, 0) > 0 and cq.workspace_bytes(-1, 5) == 0


FAKE = C.c_void_p(0x1000)      # never dereferenced: every call below fails validation first


def _act(lib, X=FAKE, dtype=1, T=16, I=64, ld=64, alpha=0.15, bits=8, deq_dtype=1, ws=FAKE, ws_bytes=1 << 30,
         codes=FAKE, deq=FAKE, zc=FAKE):
    return lib.cq_quantize_act(X, dtype, T, I, ld, alpha, bits, None, None, None, None, codes, deq, deq_dtype, zc,
                               ws, ws_bytes, None)


def test_quantize_act_rejects_bad_arguments_without_launching(lib):
    assert _act(lib, X=None) == 1                      # CQ_ERR_NULL
    assert _act(lib, T=-1) == 2                        # CQ_ERR_SHAPE
    assert _act(lib, ld=63) == 2
    assert _act(lib, dtype=2) == 3                     # CQ_ERR_DTYPE (fp32 input)
    assert _act(lib, deq_dtype=0) == 3                 # fp16 output for a bf16 input
    assert _act(lib, bits=3) == 4                      # CQ_ERR_BITS
    assert _act(lib, bits=16) == 4
    assert _act(lib, alpha=-0.01) == 5                 # CQ_ERR_ALPHA
    assert _act(lib, alpha=1.01) == 5
    assert _act(lib, alpha=float("nan")) == 5
    assert _act(lib, I=63, ld=63, bits=4) == 6         # CQ_ERR_ALIGN: odd I with INT4
    assert _act(lib, X=C.c_void_p(0x1001)) == 6        # pointer not 2-byte aligned
    assert _act(lib, zc=C.c_void_p(0x1004)) == 6
    assert _act(lib, ws=None) == 7                     # CQ_ERR_WORKSPACE
    assert _act(lib, ws=C.c_void_p(0x1010)) == 7       # not 256-byte aligned
    assert _act(lib, ws_bytes=64) == 7                 # too small


def test_other_entry_points_reject_bad_arguments(lib):
    assert lib.cq_absmax_rows(None, 1, 4, 8, 8, FAKE, None) == 1
    assert lib.cq_absmax_rows(FAKE, 1, 4, 8, 8, None, None) == 1
    assert lib.cq_absmax_cols(FAKE, 5, 4, 8, 8, FAKE, None) == 3
    assert lib.cq_absmax_rows_cols(FAKE, 1, 4, 8, 4, FAKE, FAKE, None) == 2
    assert lib.cq_dequantize(FAKE, 5, 4, 8, FAKE, FAKE, FAKE, 2, None) == 4
    assert lib.cq_dequantize(FAKE, 8, 4, 8, FAKE, FAKE, FAKE, 7, None) == 3
    assert lib.cq_dequantize(FAKE, 4, 4, 7, FAKE, FAKE, FAKE, 2, None) == 6
    assert lib.cq_dequantize(None, 8, 4, 8, FAKE, FAKE, FAKE, 2, None) == 1
    assert lib.cq_kernel_count(FAKE, 8, 4, 8, None, None) == 1
    assert lib.cq_kernel_count(FAKE, 2, 4, 8, FAKE, None) == 4
    assert lib.cq_kernel_count_x(FAKE, 1, 4, 8, 8, 0.15, 8, None, FAKE, FAKE, FAKE, 1 << 20, None) == 1
    assert lib.cq_quantize_weight_per_channel(FAKE, 1, 4, 8, 8, 5, FAKE, FAKE, None, 1, None, None) == 4
    assert lib.cq_quantize_weight_per_channel(FAKE, 1, 4, 7, 7, 4, FAKE, FAKE, None, 1, None, None) == 6
    assert lib.cq_quantize_weight_per_channel(None, 1, 4, 8, 8, 8, FAKE, FAKE, None, 1, None, None) == 1
    assert lib.cq_quantize_act_host(FAKE, 1, 4, 8, 8, 0.15, 8, None, None, None, None, None, None, 1, None, None, 0,
                                    None) == 7
    # far beyond the built-in scratch of the no-allocation entry point: refused before any CUDA call
    assert lib.cq_quantize_act_noalloc(FAKE, 1, 1 << 24, 4096, 4096, 0.15, 8, None, None, None, None, FAKE, None, 1,
                                       None, None) == 9
    assert lib.cq_set_tuning(b"no_such_knob", 4) == 2
    assert lib.cq_set_tuning(b"k3_ctas_per_sm", 0) == 0
    assert lib.cq_set_tuning(b"k3_ctas_per_sm", 1000) == 2


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2410_07505_b200 import cq
    monkeypatch.setattr(cq, "_lib", None)
    monkeypatch.setattr(cq, "LIB_PATH", str(tmp_path / "libcq.so"))
    with pytest.raises(FileNotFoundError):
        cq.lib()


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2410_07505_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
