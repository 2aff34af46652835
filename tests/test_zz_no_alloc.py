"""cq_quantize_act_noalloc -- the entry point for callers that cannot allocate device memory -- must
give exactly what cq_quantize_act gives, call after call.

Some users of the library run where cudaMalloc is off limits (all GPU memory already belongs to one
pool, or the host application bans allocation on its hot path), so this entry point keeps its scratch
in a fixed array inside the library.  Every call reuses that array and finds the previous call's
contents in it; the test therefore runs each case twice in a row, and on different shapes back to back,
and compares every output bit for bit with the ordinary entry point (the tolerance the other parity
tests use for identical arithmetic); one case is also checked against the CPU oracle directly, and the
amount of free device memory must not move across the calls.  The outputs sit between guard bands
(tests/guards.py).  The file name makes pytest collect it last.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import parity
from paper_2410_07505_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TORCH_DT = {"f16": torch.float16, "bf16": torch.bfloat16}


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
        del ref, out


def test_noalloc_matches_the_oracle_and_allocates_nothing(cq):
    T, I, dtype, bits, alpha = 515, 2056, "bf16", 8, 0.15
    X = wl.small_matrix(T, I, dtype, 4242, outlier_cols=3, zero_frac=0.01)
    Xd = _dev(X, dtype)
    out = cq.ActBuffers(T, I, Xd.dtype, bits)
    L = cq.lib()
    args = (cq._ptr(Xd), cq._DT[Xd.dtype], T, I, I, alpha, bits, cq._ptr(out.t), cq._ptr(out.c), cq._ptr(out.row_scale),
            cq._ptr(out.col_scale), cq._ptr(out.codes), cq._ptr(out.deq), cq._DT[Xd.dtype], cq._ptr(out.zero_count), None)
    assert L.cq_quantize_act_noalloc(*args) == 0           # the first call on this device may look the array up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):                                     # straight through the C ABI: no torch allocation in between
        assert L.cq_quantize_act_noalloc(*args) == 0
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0, "free device memory changed across a no-allocation call"
    out.arena.check("cq_quantize_act_noalloc")
    parity.check_act(X, dtype, alpha, bits, t=out.t.cpu().numpy(), c=out.c.cpu().numpy(), a=out.row_scale.cpu().numpy(),
                     b=out.col_scale.cpu().numpy(), codes=out.codes.cpu().numpy(),
                     deq=out.deq.view(torch.int16).cpu().numpy().view(np.uint16), zero_count=int(out.zero_count.item()))


def test_noalloc_refuses_shapes_beyond_its_scratch(cq):
    T, I = 3_000_000, 8                                             # three fp32 vectors of 12 MB alone exceed 8 MiB
    assert cq.workspace_bytes(T, I) > cq.NOALLOC_SCRATCH_BYTES
    Xd = torch.zeros((T, I), dtype=torch.bfloat16, device="cuda")
    out = cq.ActBuffers(T, I, torch.bfloat16, 8)
    with pytest.raises(cq.CQError) as e:
        cq.quantize_act_noalloc(Xd, 0.15, 8, buffers=out)
    assert e.value.status == 9
    assert "scratch" in str(e.value)
