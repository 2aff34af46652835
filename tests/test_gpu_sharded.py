"""One matrix in several row blocks (the exchange step of a token-sharded or streamed X): the blocks'
results, put together, must equal the oracle's on the whole matrix."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import parity
from paper_2410_07505_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TORCH_DT = {"f16": torch.float16, "bf16": torch.bfloat16}


@pytest.fixture(scope="module")
def mods(cq):
    """(binding behind guard bands, the sharded module made to allocate and call through the same guarded binding)."""
    from paper_2410_07505_b200 import sharded
    plain = sharded.cq
    sharded.cq = cq
    yield cq, sharded
    sharded.cq = plain


def to_dev(bits: np.ndarray, dtype: str) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(TORCH_DT[dtype]).cuda()


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def check_blocks(X, dtype, alpha, bits, outs, total):
    T, I = X.shape
    parity.check_act(X, dtype, alpha, bits,
                     t=np.concatenate([o.t.cpu().numpy() for o in outs]),
                     c=outs[0].c.cpu().numpy(),
                     a=np.concatenate([o.row_scale.cpu().numpy() for o in outs]),
                     b=outs[0].col_scale.cpu().numpy(),
                     codes=np.concatenate([o.codes.cpu().numpy().reshape(o.t.numel(), -1) for o in outs]),
                     deq=np.concatenate([bits_of(o.deq).reshape(o.t.numel(), I) for o in outs]),
                     zero_count=int(total))
    for o in outs[1:]:                                       # every block used the same column vectors
        assert torch.equal(o.c, outs[0].c) and torch.equal(o.col_scale, outs[0].col_scale)


@pytest.mark.parametrize("shape,cuts", [((301, 1000), (100, 157)), ((64, 2056), (1, 63)), ((50, 77), (20, 21)),
                                         ((1030, 4104), (512, 1024))])
@pytest.mark.parametrize("dtype,bits,alpha", [("f16", 8, 0.15), ("bf16", 4, 0.5), ("bf16", 8, 0.0), ("f16", 8, 1.0)])
def test_row_chunks_equal_the_whole_matrix(mods, shape, cuts, dtype, bits, alpha):
    cq, sharded = mods
    T, I = shape
    if bits == 4 and I % 2:
        pytest.skip("INT4 packs two columns per byte")
    X = wl.small_matrix(T, I, dtype, 300 + T + I, outlier_cols=3, zero_frac=0.02)
    Xd = to_dev(X, dtype)
    chunks = [Xd[0:cuts[0]], Xd[cuts[0]:cuts[1]], Xd[cuts[1]:T]]
    outs, total = sharded.quantize_act_chunked(chunks, alpha, bits)
    torch.cuda.synchronize()
    check_blocks(X, dtype, alpha, bits, outs, total)


def test_running_column_maximum_is_the_column_absmax(mods):
    cq, _ = mods
    X = wl.small_matrix(200, 520, "bf16", 5, outlier_cols=4)
    Xd = to_dev(X, "bf16")
    _, c_full = cq.absmax_rows_cols(Xd)
    _, c = cq.absmax_rows_cols(Xd[:70])
    for r0, r1 in ((70, 71), (71, 200)):
        cq.vector_max_(c, cq.absmax_rows_cols(Xd[r0:r1])[1])
    assert torch.equal(c, c_full)


def test_row_sharded_call_on_one_rank_equals_the_plain_call(mods):
    cq, sharded = mods
    X = wl.small_matrix(130, 2056, "f16", 9, outlier_cols=2, zero_frac=0.01)
    Xd = to_dev(X, "f16")
    out, total = sharded.quantize_act_row_sharded(Xd, 0.15, 8)              # no process group: a world of one
    torch.cuda.synchronize()
    check_blocks(X, "f16", 0.15, 8, [out], int(total.item()))


def test_given_maxima_full_size_sample(mods):
    """Headline shape in two halves: rows sampled from both halves against the oracle's whole-matrix result."""
    cq, sharded = mods
    from oracle import cq_oracle as orc
    X, cfg = wl.activation("llama70b_attn")
    Xd = to_dev(X, cfg.dtype)
    half = cfg.T // 2
    outs, total = sharded.quantize_act_chunked([Xd[:half], Xd[half:]], 0.15, 8)
    torch.cuda.synchronize()
    ref = orc.quantize_act(X, cfg.dtype, 0.15, 8, want_deq16=True)
    assert total == int(ref.zero_count)
    rows = np.array([0, 1, half - 1, half, half + 1, cfg.T - 1, 777, 3001])
    got = np.concatenate([o.codes.cpu().numpy() for o in outs])[rows]
    assert np.array_equal(got.view(np.int8), ref.codes[rows])
    assert np.array_equal(outs[0].c.cpu().numpy().view(np.uint32), ref.c.view(np.uint32))


@pytest.mark.parametrize("shape", [(130, 2056), (33, 50), (1, 8)])
def test_absmax_with_a_workspace_equals_the_atomic_entry_point(mods, shape):
    cq, _ = mods
    X = wl.small_matrix(shape[0], shape[1], "bf16", 21, outlier_cols=2, zero_frac=0.05)
    Xd = to_dev(X, "bf16")
    ws = torch.empty(cq.workspace_bytes(*shape), dtype=torch.uint8, device="cuda")
    t0, c0 = cq.absmax_rows_cols(Xd)
    t1, c1 = cq.absmax_rows_cols(Xd, workspace=ws)
    assert torch.equal(t0, t1) and torch.equal(c0, c1)


@pytest.mark.parametrize("shape,cuts", [((130, 2056), (1024, 1544)), ((64, 4104), (8, 2056)), ((37, 90), (30, 31))])
@pytest.mark.parametrize("dtype,bits,alpha", [("bf16", 8, 0.15), ("f16", 4, 0.5), ("bf16", 8, 1.0)])
def test_column_blocks_equal_the_whole_matrix(mods, shape, cuts, dtype, bits, alpha):
    cq, sharded = mods
    T, I = shape
    if bits == 4 and any(c % 2 for c in cuts):
        pytest.skip("INT4 packs two columns per byte")
    X = wl.small_matrix(T, I, dtype, 500 + T + I, outlier_cols=3, zero_frac=0.02)
    Xd = to_dev(X, dtype)
    blocks = [Xd[:, 0:cuts[0]], Xd[:, cuts[0]:cuts[1]], Xd[:, cuts[1]:I]]        # views: rows I elements apart
    outs, total = sharded.quantize_act_column_blocks(blocks, alpha, bits)
    torch.cuda.synchronize()
    from oracle import cq_oracle as orc
    ref = orc.quantize_act(X, dtype, alpha, bits, want_deq32=False, want_deq16=True)
    assert total == int(ref.zero_count)
    edges = [0, cuts[0], cuts[1], I]
    for o, j0, j1 in zip(outs, edges[:-1], edges[1:]):
        assert np.array_equal(o.t.cpu().numpy().view(np.uint32), ref.t.view(np.uint32))
        assert np.array_equal(o.c.cpu().numpy().view(np.uint32), ref.c[j0:j1].view(np.uint32))
        codes = o.codes.cpu().numpy()
        codes = parity.unpack_int4(codes, T, j1 - j0) if bits == 4 else codes.view(np.int8)
        assert np.array_equal(codes, ref.codes[:, j0:j1])
        assert np.array_equal(bits_of(o.deq).reshape(T, j1 - j0), ref.deq16[:, j0:j1])


def test_block_entry_points_report_bad_arguments(mods):
    cq, _ = mods
    L = cq.lib()
    X = to_dev(wl.small_matrix(8, 64, "bf16", 1), "bf16")
    ws = torch.empty(cq.workspace_bytes(8, 64), dtype=torch.uint8, device="cuda")
    v = torch.ones(64, dtype=torch.float32, device="cuda")
    assert L.cq_vector_max(None, None, 0, None) == 0                     # nothing to do
    assert L.cq_vector_max(None, cq._ptr(v), 64, None) == 1              # CQ_ERR_NULL
    assert L.cq_vector_max(cq._ptr(v), cq._ptr(v), -1, None) == 2        # CQ_ERR_SHAPE
    rc = L.cq_quantize_act_given(cq._ptr(X), 1, 8, 64, 64, 0.15, 8, None, cq._ptr(v), None, None, None, None, 1, None,
                                 cq._ptr(ws), ws.numel(), None)
    assert rc == 1                                                       # t missing
    rc = L.cq_quantize_act_given(cq._ptr(X), 1, 8, 64, 64, 1.5, 8, cq._ptr(v), cq._ptr(v), None, None, None, None, 1, None,
                                 cq._ptr(ws), ws.numel(), None)
    assert rc == 5                                                       # alpha out of range
    with pytest.raises(ValueError):
        cq.vector_max_(v, v[:32])
    torch.cuda.synchronize()


def test_an_empty_row_block_contributes_zeros_to_the_combined_maxima(mods):
    """A rank or chunk without rows (T < world size) still hands a column-maximum vector to the exchange: it must be
    zeros, whatever the buffer held before, and the other blocks' results must equal the whole matrix's."""
    cq, sharded = mods
    X = wl.small_matrix(5, 264, "bf16", 17, outlier_cols=2)
    Xd = to_dev(X, "bf16")
    b = cq.ActBuffers(0, 264, Xd.dtype, 8)
    b.c.fill_(float("nan"))
    b.col_scale.fill_(float("nan"))
    _, c = cq.absmax_rows_cols(Xd[0:0], workspace=b.workspace, out=(b.t, b.c))
    torch.cuda.synchronize()
    assert not c.any() and c.numel() == 264
    r = cq.quantize_act(Xd[0:0], 0.15, 8, buffers=b)                        # scale factors of c = 0: zeros too
    assert int(r.zero_count.item()) == 0 and not r.col_scale.any()
    for alpha in (0.15, 1.0):
        outs, total = sharded.quantize_act_chunked([Xd[:3], Xd[3:3], Xd[3:]], alpha, 8)
        torch.cuda.synchronize()
        assert torch.equal(outs[1].c, outs[0].c)
        check_blocks(X, "bf16", alpha, 8, [outs[0], outs[2]], total)
    # the same for a column block without columns: its row maxima are zeros
    b = cq.ActBuffers(5, 0, Xd.dtype, 8)
    b.t.fill_(float("nan"))
    t, _ = cq.absmax_rows_cols(Xd[:, 0:0], workspace=b.workspace, out=(b.t, b.c))
    assert not t.any() and t.numel() == 5
