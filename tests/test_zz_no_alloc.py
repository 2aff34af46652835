"""cq_quantize_act_noalloc -- the entry point for callers that cannot allocate device memory -- must
give exactly what cq_quantize_act gives, call after call.

Some users of the library run where cudaMalloc is off limits (all GPU memory already belongs to one
pool, or the host application bans allocation on its hot path), so this entry point keeps its scratch
in a fixed array inside the library.  Every call reuses that array and finds the previous call's
contents in it; the test therefore runs each case twice in a row, and on different shapes back to back,
and compares every output bit for bit with the ordinary entry point (the tolerance the other parity
tests use for identical arithmetic).  The file name makes pytest collect it last.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from paper_2410_07505_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TORCH_DT = {"f16": torch.float16, "bf16": torch.bfloat16}


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2410_07505_b200 import build, cq as _cq
    build.build()
    _cq.lib()
    return _cq


def _dev(bits, dtype):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(TORCH_DT[dtype]).cuda()


def _same(r, ref):
    for name in ("t", "c", "row_scale", "col_scale", "codes", "zero_count"):
        assert torch.equal(getattr(r, name), getattr(ref, name)), name
    assert torch.equal(r.deq.view(torch.int16), ref.deq.view(torch.int16)), "deq"


CASES = [(300, 1536, "bf16", 8, 0.15), (128, 768, "f16", 4, 0.5), (1024, 8192, "bf16", 8, 0.15),
         (33, 50, "f16", 8, 0.15), (2048, 28672, "bf16", 4, 0.15)]


def test_noalloc_matches_the_ordinary_entry_point_on_repeated_calls(cq):
    for T, I, dtype, bits, alpha in CASES:
        X = wl.small_matrix(T, I, dtype, 900 + T, outlier_cols=3, zero_frac=0.01)
        Xd = _dev(X, dtype)
        ref = cq.quantize_act(Xd, alpha, bits)                      # ordinary entry point, caller's workspace
        out = cq.ActBuffers(T, I, Xd.dtype, bits)                   # outputs only; its workspace stays unused
        for call in range(2):                                       # two calls in a row on the shared scratch
            for buf in (out.t, out.c, out.row_scale, out.col_scale, out.codes, out.deq):
                buf.fill_(1)                                        # stale outputs must be overwritten
            r = cq.quantize_act_noalloc(Xd, alpha, bits, buffers=out)
            torch.cuda.synchronize()
            _same(r, ref)


def test_noalloc_refuses_shapes_beyond_its_scratch(cq):
    T, I = 3_000_000, 8                                             # three fp32 vectors of 12 MB alone exceed 8 MiB
    assert cq.workspace_bytes(T, I) > cq.NOALLOC_SCRATCH_BYTES
    Xd = torch.zeros((T, I), dtype=torch.bfloat16, device="cuda")
    out = cq.ActBuffers(8, 8, torch.bfloat16, 8)
    with pytest.raises(cq.CQError) as e:
        cq.quantize_act_noalloc(Xd, 0.15, 8, buffers=out)
    assert e.value.status == 9
    assert "scratch" in str(e.value)
