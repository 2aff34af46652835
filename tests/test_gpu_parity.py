"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import cq_oracle as orc
from oracle import parity
from paper_2410_07505_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TORCH_DT = {"f16": torch.float16, "bf16": torch.bfloat16}


def to_dev(bits: np.ndarray, dtype: str) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(TORCH_DT[dtype]).cuda()


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def run_and_check(cq, X, dtype, alpha, bits, *, deq_f32=False, Xd=None, ref=None):
    Xd = to_dev(X, dtype) if Xd is None else Xd
    r = cq.quantize_act(Xd, alpha, bits, deq_dtype=torch.float32 if deq_f32 else None)
    torch.cuda.synchronize()
    deq = r.deq.cpu().numpy() if deq_f32 else bits_of(r.deq)
    return parity.check_act(X, dtype, alpha, bits, t=r.t.cpu().numpy(), c=r.c.cpu().numpy(),
                            a=r.row_scale.cpu().numpy(), b=r.col_scale.cpu().numpy(),
                            codes=r.codes.cpu().numpy(), deq=deq, deq_is_f32=deq_f32,
                            zero_count=int(r.zero_count.item()), ref=ref), r


# ------------------------------------------------------------------ small, multi-tile, ragged
FAST_SHAPES = [(1, 8), (3, 16), (37, 264), (130, 2056), (257, 776), (64, 4104), (19, 2048)]
GENERAL_SHAPES = [(1, 1), (5, 7), (33, 50), (17, 1001), (70, 258)]


@pytest.mark.parametrize("shape", FAST_SHAPES + GENERAL_SHAPES)
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_small_shapes_all_alphas_and_bit_widths(cq, shape, dtype):
    T, I = shape
    X = wl.small_matrix(T, I, dtype, 1000 + T + I, outlier_cols=2, zero_frac=0.01)
    for bits in (8, 4):
        if bits == 4 and I % 2:
            continue
        for alpha in (0.0, 0.15, 0.5, 1.0):
            rep, _ = run_and_check(cq, X, dtype, alpha, bits)
            assert rep.scales_identical and rep.code_mismatches == 0
    rep, _ = run_and_check(cq, X, dtype, 0.15, 8, deq_f32=True)
    assert rep.max_deq_ulp == 0


@pytest.mark.parametrize("dist", ["student_t3", "laplace"])
def test_heavy_tailed_values(cq, dist):
    X = wl.small_matrix(300, 1536, "bf16", 77, dist=dist, outlier_cols=5, outlier_scale=50.0)
    for alpha in (0.15, 0.45, 0.75):
        for bits in (8, 4):
            run_and_check(cq, X, "bf16", alpha, bits)


def test_leading_dimension_and_offset_views(cq):
    big = wl.small_matrix(90, 640, "bf16", 5)
    bd = to_dev(big, "bf16")
    # aligned window: fast kernels with ld > I
    win = np.ascontiguousarray(big[:, 64:64 + 256])
    run_and_check(cq, win, "bf16", 0.15, 8, Xd=bd[:, 64:64 + 256])
    run_and_check(cq, win, "bf16", 0.5, 4, Xd=bd[:, 64:64 + 256])
    # odd offset: pointer only 2-byte aligned -> general kernels
    win = np.ascontiguousarray(big[:, 3:3 + 250])
    run_and_check(cq, win, "bf16", 0.15, 8, Xd=bd[:, 3:3 + 250])
    run_and_check(cq, win, "bf16", 0.15, 4, Xd=bd[:, 3:3 + 250])


def test_empty_matrices(cq):
    for T, I in [(0, 64), (16, 0), (0, 0)]:
        Xd = torch.empty((T, I), dtype=torch.float16, device="cuda")
        r = cq.quantize_act(Xd, 0.15, 8)
        torch.cuda.synchronize()
        assert int(r.zero_count.item()) == 0
        assert cq.absmax_rows(Xd).shape == (T,) and cq.absmax_cols(Xd).shape == (I,)
        if T == 0 and I > 0:
            assert not cq.absmax_cols(Xd).any()


@pytest.mark.parametrize("alpha", [0.0, 0.15, 1.0])
def test_zero_row_zero_column_and_all_zero(cq, alpha):
    X = wl.small_matrix(40, 128, "bf16", 9, outlier_cols=0)
    X[7, :] = 0
    X[:, 11] = 0x8000
    rep, r = run_and_check(cq, X, "bf16", alpha, 8, deq_f32=True)
    assert torch.isfinite(r.deq).all()
    assert not r.codes[7].any() and not r.codes[:, 11].any()
    Z = np.zeros((16, 64), dtype=np.uint16)
    rep, r = run_and_check(cq, Z, "f16", alpha, 4)
    assert rep.zero_count == 16 * 64


def test_extreme_magnitudes(cq):
    # largest fp16 values
    X = wl.small_matrix(32, 256, "f16", 3, scale=300.0, outlier_cols=2, outlier_scale=20.0)
    assert np.isfinite(wl.bits_to_f32(X, "f16")).all()
    X[0, 0] = 0x7BFF
    X[5, 9] = 0xFBFF
    run_and_check(cq, X, "f16", 0.15, 8)
    run_and_check(cq, X, "f16", 0.15, 8, deq_f32=True)
    # fp16 subnormals only
    S = (np.arange(32 * 64, dtype=np.uint16).reshape(32, 64) % 1024)
    S[1::2] |= 0x8000
    run_and_check(cq, S, "f16", 0.5, 8)
    # bf16 near the top and the bottom of the fp32 exponent range (scales become subnormal)
    for scale in (1e36, 1e-36, 3e-39):
        B = wl.small_matrix(24, 128, "bf16", 4, scale=scale, outlier_cols=1, outlier_scale=8.0)
        for alpha in (0.0, 0.15, 0.5, 1.0):
            run_and_check(cq, B, "bf16", alpha, 8, deq_f32=True)
            run_and_check(cq, B, "bf16", alpha, 4)


def test_exact_ties_round_to_even_on_the_gpu(cq):
    row = np.zeros((1, 16), dtype=np.float32)
    row[0, :10] = [127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 126.5, -125.5]
    X = wl.to_bits(row, "f16")
    rep, r = run_and_check(cq, X, "f16", 1.0, 8)
    assert r.codes[0, :10].tolist() == [127, 0, 2, 2, 0, -2, -2, 4, 126, -126]


def test_outputs_are_optional(cq):
    X = wl.small_matrix(65, 512, "bf16", 12)
    Xd = to_dev(X, "bf16")
    ref = orc.quantize_act(X, "bf16", 0.15, 8)
    r = cq.quantize_act(Xd, 0.15, 8, codes=False, deq=False)
    assert int(r.zero_count.item()) == ref.zero_count
    r = cq.quantize_act(Xd, 0.15, 8, codes=True, deq=False, count=False)
    assert np.array_equal(r.codes.cpu().numpy(), ref.codes)
    r = cq.quantize_act(Xd, 0.15, 8, codes=False, deq=True, count=False)
    assert np.array_equal(bits_of(r.deq), ref.deq16)


def test_tiling_knobs_do_not_change_results(cq):
    X = wl.small_matrix(333, 2304, "bf16", 13, outlier_cols=3)
    ref = orc.quantize_act(X, "bf16", 0.15, 8)
    try:
        for k1, k3, fwd in [(1, 1, 0), (2, 5, 1), (8, 2, 0), (3, 64, 1)]:
            cq.set_tuning("k1_ctas_per_sm", k1)
            cq.set_tuning("k3_ctas_per_sm", k3)
            cq.set_tuning("k3_forward", fwd)
            run_and_check(cq, X, "bf16", 0.15, 8, ref=ref)
    finally:
        for key in ("k1_ctas_per_sm", "k3_ctas_per_sm", "k3_forward"):
            cq.set_tuning(key, 0)


SMALL_SHAPES = [(1, 8), (1, 4096), (3, 16), (16, 4096), (16, 8192), (32, 2048), (31, 776), (9, 5000), (5, 8200), (16, 6152),
                (33, 2048), (17, 8192),
                # narrow strips hold more rows per cluster CTA (up to 16, up to 1024 vectors per tile); one or two strips
                # may take a 16-CTA cluster: shapes at and just past those limits
                (128, 768), (129, 768), (256, 256), (250, 200), (257, 256), (64, 2048), (65, 2048), (32, 4096), (33, 4096),
                (160, 512), (161, 520)]


@pytest.mark.parametrize("shape", SMALL_SHAPES)
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_small_matrices_one_launch_and_three_launches(cq, shape, dtype):
    """Decode-sized matrices take a single thread-block-cluster launch (4 rows of a full strip to 16 rows of a narrow one
    per cluster CTA, up to four column strips); the shapes around its limits and the same shapes forced through the
    three launches."""
    T, I = shape
    X = wl.small_matrix(T, I, dtype, 700 + T + I, outlier_cols=3, outlier_scale=30.0, zero_frac=0.03)
    X[0, : min(I, 24)] = 0
    Xd = to_dev(X, dtype)
    try:
        for no_small in (0, 1):
            cq.set_tuning("no_small", no_small)
            for alpha, bits in [(0.15, 8), (0.5, 4), (1.0, 8), (0.0, 4)]:
                if bits == 4 and I % 2:
                    continue
                run_and_check(cq, X, dtype, alpha, bits, Xd=Xd)
            run_and_check(cq, X, dtype, 0.15, 8, deq_f32=True, Xd=Xd)
            r = cq.quantize_act(Xd, 0.15, 8, codes=False, deq=False)          # count only
            assert int(r.zero_count.item()) == orc.quantize_act(X, dtype, 0.15, 8, want_deq32=False, want_deq16=False).zero_count
    finally:
        cq.set_tuning("no_small", 0)
    assert cq.stage_fault() == 0


@pytest.mark.parametrize("shape", [(300, 2056), (16, 4096), (513, 776)])
def test_public_call_replays_from_a_cuda_graph(cq, shape):
    """After one ordinary call (which settles the per-kernel launch attributes) the call only enqueues kernels,
    so it can be captured once and replayed on new contents of the same buffers."""
    T, I = shape
    X1 = wl.small_matrix(T, I, "bf16", 31, outlier_cols=3, zero_frac=0.02)
    X2 = wl.small_matrix(T, I, "bf16", 32, outlier_cols=3, zero_frac=0.02)
    Xd = to_dev(X1, "bf16")
    buf = cq.ActBuffers(T, I, Xd.dtype, 8)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        cq.quantize_act(Xd, 0.15, 8, buffers=buf)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        cq.quantize_act(Xd, 0.15, 8, buffers=buf)
    for X in (X1, X2, X1):
        Xd.copy_(to_dev(X, "bf16"))
        for b in (buf.codes, buf.deq, buf.t, buf.c, buf.row_scale, buf.col_scale):
            b.zero_()
        graph.replay()
        torch.cuda.synchronize()
        buf.arena.check("graph replay")
        parity.check_act(X, "bf16", 0.15, 8, t=buf.t.cpu().numpy(), c=buf.c.cpu().numpy(), a=buf.row_scale.cpu().numpy(),
                         b=buf.col_scale.cpu().numpy(), codes=buf.codes.cpu().numpy(), deq=bits_of(buf.deq),
                         zero_count=int(buf.zero_count.item()))


def test_launch_without_programmatic_dependent_launch_gives_the_same_results(cq):
    try:
        cq.set_tuning("no_pdl", 1)
        for (T, I), dtype in [((130, 2056), "bf16"), ((257, 776), "f16"), ((1027, 4104), "f16")]:
            X = wl.small_matrix(T, I, dtype, 3000 + T, outlier_cols=2, zero_frac=0.01)
            for bits, alpha in [(8, 0.15), (4, 0.5)]:
                run_and_check(cq, X, dtype, alpha, bits)
    finally:
        cq.set_tuning("no_pdl", 0)


def test_tall_and_wide_extremes(cq):
    # many more row groups than resident CTAs, and a single group
    for T, I in [(5000, 64), (20000, 8), (2, 16384), (4, 40000)]:
        X = wl.small_matrix(T, I, "f16", 15, outlier_cols=1)
        run_and_check(cq, X, "f16", 0.15, 8)
        run_and_check(cq, X, "f16", 0.5, 4)
    # more than 65,535 blocks of 64 rows through the general (unaligned) kernels: their grids are one-dimensional
    X = wl.small_matrix(4_200_000, 2, "bf16", 16, outlier_cols=1)
    run_and_check(cq, X, "bf16", 0.15, 8)
    run_and_check(cq, X, "bf16", 0.5, 4)


def test_repeated_calls_reuse_buffers(cq):
    X = wl.small_matrix(128, 1024, "f16", 14)
    Xd = to_dev(X, "f16")
    buf = cq.ActBuffers(128, 1024, torch.float16, 8)
    ref = orc.quantize_act(X, "f16", 0.15, 8)
    for _ in range(3):
        r = cq.quantize_act(Xd, 0.15, 8, buffers=buf)
        assert int(r.zero_count.item()) == ref.zero_count
        assert np.array_equal(r.codes.cpu().numpy(), ref.codes)


# ------------------------------------------------------------------ the other entry points
@pytest.mark.parametrize("shape,dtype", [((130, 2056), "bf16"), ((33, 50), "f16"), ((1, 8), "f16"), ((700, 96), "bf16")])
def test_absmax_entry_points(cq, shape, dtype):
    X = wl.small_matrix(*shape, dtype, 21)
    Xd = to_dev(X, dtype)
    t_ref, c_ref = orc.absmax_rows(X, dtype), orc.absmax_cols(X, dtype)
    t, c = cq.absmax_rows_cols(Xd)
    assert np.array_equal(t.cpu().numpy(), t_ref) and np.array_equal(c.cpu().numpy(), c_ref)
    assert np.array_equal(cq.absmax_rows(Xd).cpu().numpy(), t_ref)
    assert np.array_equal(cq.absmax_cols(Xd).cpu().numpy(), c_ref)


# (262147, 8): more groups of four rows than a grid may have in y (the kernel loops); (7, 4104): three blocks of vector
# columns, the last one ragged, and a ragged last row group
@pytest.mark.parametrize("shape", [(65, 512), (33, 50), (9, 1030), (262147, 8), (7, 4104)])
@pytest.mark.parametrize("bits", [8, 4])
def test_dequantize_and_kernel_count_from_stored_codes(cq, shape, bits):
    T, I = shape
    X = wl.small_matrix(T, I, "bf16", 31, zero_frac=0.02)
    ref = orc.quantize_act(X, "bf16", 0.15, bits)
    stored = ref.codes if bits == 8 else ref.packed_int4()
    cd = torch.from_numpy(stored).cuda()
    a, b = torch.from_numpy(ref.a).cuda(), torch.from_numpy(ref.b).cuda()
    out32 = cq.dequantize(cd, bits, T, I, a, b, torch.float32).cpu().numpy()
    assert np.array_equal(out32.view(np.uint32), ref.deq32.view(np.uint32))
    out16 = cq.dequantize(cd, bits, T, I, a, b, torch.bfloat16)
    assert np.array_equal(bits_of(out16), ref.deq16)
    outh = cq.dequantize(cd, bits, T, I, a, b, torch.float16)
    assert np.array_equal(bits_of(outh), orc.encode16(ref.deq32, "f16"))
    assert int(cq.kernel_count(cd, bits, T, I).item()) == ref.zero_count
    # misaligned start of the code buffer
    if bits == 8:
        pad = torch.zeros(stored.size + 3, dtype=torch.int8, device="cuda")
        pad[3:] = cd.flatten()
        assert int(cq.kernel_count(pad[3:], bits, T, I).item()) == ref.zero_count


def test_dequantize_more_row_groups_than_grid_rows(cq):
    """262,150 rows of 1032 codes: 65,538 groups of four rows, more than a grid may have in y, so the kernel loops.
    Row blocks of the result (the first, one across the grid limit, the ragged last) must equal what separate calls
    on those rows alone give (small calls of this kind are compared with the oracle above)."""
    T, I = 262150, 1032
    g = torch.Generator(device="cuda").manual_seed(5)
    codes = torch.randint(-127, 128, (T, I), dtype=torch.int8, device="cuda", generator=g)
    a = torch.rand(T, device="cuda", generator=g) + 0.01
    b = torch.rand(I, device="cuda", generator=g) + 0.01
    out = cq.dequantize(codes, 8, T, I, a, b, torch.bfloat16)
    for lo, hi in ((0, 9), (4 * 65535 - 3, 4 * 65535 + 5), (T - 6, T)):
        part = cq.dequantize(codes[lo:hi].contiguous(), 8, hi - lo, I, a[lo:hi].contiguous(), b, torch.bfloat16)
        assert torch.equal(out[lo:hi].view(torch.int16), part.view(torch.int16))
    assert int(cq.kernel_count(codes, 8, T, I).item()) == int((codes == 0).sum().item())


@pytest.mark.parametrize("bits", [8, 4])
def test_kernel_count_straight_from_x(cq, bits):
    X = wl.small_matrix(200, 1032, "f16", 41, outlier_cols=4, outlier_scale=40.0, zero_frac=0.01)
    Xd = to_dev(X, "f16")
    t, c = cq.absmax_rows_cols(Xd)
    for alpha in (0.15, 1.0):
        ref = orc.quantize_act(X, "f16", alpha, bits, want_deq32=False, want_deq16=False)
        assert int(cq.kernel_count_x(Xd, alpha, bits, t, c).item()) == ref.zero_count


WEIGHT_SHAPES = [(1, 8), (5, 264), (40, 2056), (7, 8192), (3, 28672), (33, 50), (6, 1001), (2, 110600), (5, 12296),
                 (3, 57352), (2, 300000)]


@pytest.mark.parametrize("shape", WEIGHT_SHAPES)
@pytest.mark.parametrize("bits", [8, 4])
def test_weight_per_channel(cq, shape, bits):
    R, Cc = shape
    if bits == 4 and Cc % 2:
        pytest.skip("INT4 needs an even number of columns")
    for dtype in ("bf16", "f16"):
        W = wl.small_matrix(R, Cc, dtype, 51 + R, scale=0.02, outlier_cols=1, outlier_scale=6.0)
        if R > 2:
            W[1, :] = 0
        Wd = to_dev(W, dtype)
        ref = orc.quantize_weight_per_channel(W, dtype, bits)
        r = cq.quantize_weight_per_channel(Wd, bits)
        torch.cuda.synchronize()
        parity.check_weight(W, dtype, bits, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(),
                            deq=bits_of(r.deq), zero_count=int(r.zero_count.item()), ref=ref)
        r = cq.quantize_weight_per_channel(Wd, bits, deq_dtype=torch.float32)
        parity.check_weight(W, dtype, bits, deq=r.deq.cpu().numpy(), deq_is_f32=True, ref=ref)


@pytest.mark.parametrize("shape,group", [((7, 1024), 128), ((3, 8192), 128), ((33, 256), 64), ((5, 512), 256),
                                         ((9, 96), 32), ((4, 64), 8), ((6, 240), 48), ((5, 100), 10), ((3, 1024), 1024)])
@pytest.mark.parametrize("bits", [8, 4])
def test_weight_groupwise(cq, shape, group, bits):
    R, Cc = shape
    for dtype in ("bf16", "f16"):
        W = wl.small_matrix(R, Cc, dtype, 91 + R, scale=0.02, outlier_cols=2, outlier_scale=8.0)
        W[0, :group] = 0                                     # one all-zero group
        ref = orc.quantize_weight_groupwise(W, dtype, bits, group)
        r = cq.quantize_weight_groupwise(to_dev(W, dtype), group, bits)
        torch.cuda.synchronize()
        parity.check_weight(W, dtype, bits, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(),
                            deq=bits_of(r.deq), zero_count=int(r.zero_count.item()), ref=ref)
        r = cq.quantize_weight_groupwise(to_dev(W, dtype), group, bits, deq_dtype=torch.float32)
        parity.check_weight(W, dtype, bits, deq=r.deq.cpu().numpy(), deq_is_f32=True, ref=ref)


@pytest.mark.parametrize("bits,top", [(8, 254), (4, 14)])
def test_rows_full_of_exact_ties(cq, bits, top):
    """A row maximum of 2 * qmax * 2^e puts every odd multiple of 2^e on a rounding tie (x / d = k / 2): the
    re-examination path has to settle them all to the even neighbour, for weights, groups and activations."""
    rng = np.random.Generator(np.random.PCG64(77))
    for dtype in ("bf16", "f16"):
        for e in (-10, 0, 3):
            k = rng.integers(-top, top + 1, size=(37, 1024)).astype(np.float32)
            k[:, ::128] = top                                  # every group of 128 holds the maximum
            k[5, :] = 0
            W = wl.to_bits(k * np.float32(2.0 ** e), dtype)
            assert np.array_equal(wl.bits_to_f32(W, dtype), k * np.float32(2.0 ** e))   # exactly representable
            Wd = to_dev(W, dtype)
            ref = orc.quantize_weight_per_channel(W, dtype, bits)
            r = cq.quantize_weight_per_channel(Wd, bits)
            parity.check_weight(W, dtype, bits, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(),
                                deq=bits_of(r.deq), zero_count=int(r.zero_count.item()), ref=ref)
            refg = orc.quantize_weight_groupwise(W, dtype, bits, 128)
            g = cq.quantize_weight_groupwise(Wd, 128, bits)
            parity.check_weight(W, dtype, bits, scale=g.scale.cpu().numpy(), codes=g.codes.cpu().numpy(),
                                deq=bits_of(g.deq), zero_count=int(g.zero_count.item()), ref=refg)
            run_and_check(cq, W, dtype, 1.0, bits, Xd=Wd)      # per-token activations: the same ties
            ties = np.abs(k / 2 - np.trunc(k / 2)) == 0.5
            assert ties.mean() > 0.3


@pytest.mark.parametrize("scale", [1e36, 1e-36, 3e-39, 2.0 ** -41, 2.0 ** 41])
def test_weight_scales_outside_the_exact_quotient_range(cq, scale):
    """Row and group scales beyond [2^-40, 2^40] (down to subnormal ones) leave the division-free quotient and take the
    defining sequence; rows inside the range sit next to them in the same matrix."""
    for bits in (8, 4):
        W = wl.small_matrix(12, 1024, "bf16", 63, scale=scale, outlier_cols=2, outlier_scale=4.0, zero_frac=0.02)
        W[3] = wl.small_matrix(1, 1024, "bf16", 64, scale=0.02)[0]            # an ordinary row among the extreme ones
        W[7, :] = 0
        Wd = to_dev(W, "bf16")
        ref = orc.quantize_weight_per_channel(W, "bf16", bits)
        r = cq.quantize_weight_per_channel(Wd, bits)
        parity.check_weight(W, "bf16", bits, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(), deq=bits_of(r.deq),
                            zero_count=int(r.zero_count.item()), ref=ref)
        refg = orc.quantize_weight_groupwise(W, "bf16", bits, 128)
        g = cq.quantize_weight_groupwise(Wd, 128, bits)
        parity.check_weight(W, "bf16", bits, scale=g.scale.cpu().numpy(), codes=g.codes.cpu().numpy(), deq=bits_of(g.deq),
                            zero_count=int(g.zero_count.item()), ref=refg)


def test_weight_groupwise_rejects_a_group_that_does_not_divide_the_row(cq):
    Wd = torch.zeros((4, 100), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cq.CQError) as e:
        cq.quantize_weight_groupwise(Wd, 128, 4)
    assert e.value.status == 2


@pytest.mark.parametrize("shape,dtype", [((130, 2056), "bf16"), ((37, 264), "f16"), ((33, 50), "bf16"), ((5, 7), "f16"),
                                         ((1027, 512), "bf16")])
def test_remove_kernel(cq, shape, dtype):
    T, I = shape
    X = wl.small_matrix(T, I, dtype, 97, outlier_cols=3, outlier_scale=40.0, zero_frac=0.01)
    X[3 % T, :] = 0
    Xd = to_dev(X, dtype)
    for alpha, bits, theta in [(0.15, 8, 1.0), (1.0, 8, 1.0), (0.5, 4, 1.0), (0.15, 8, 0.37), (0.15, 8, 3.0), (0.0, 8, 0.0)]:
        want, removed, k_pt, k_cq = orc.remove_kernel(X, dtype, alpha, bits, theta)
        out, counts = cq.remove_kernel(Xd, alpha, bits, theta)
        torch.cuda.synchronize()
        assert counts.cpu().tolist() == [removed, k_pt, k_cq]
        assert np.array_equal(bits_of(out), want)


def test_zero_tests_on_exact_boundaries_and_extreme_scales(cq):
    """The diagnostics kernel decides |fl32(x/s)| <= h from products and thresholds; the cases it must hand
    to the quotient: elements exactly on the bound, neighbours of the bound, scales and bounds outside
    the range the shortcut covers."""
    # per-token rows with s_i = 2^k: x = s/2 is exactly on the bound 1/2 (code 0 by round-half-even)
    rows = []
    for k in (-6, 0, 5):
        s = np.float32(2.0 ** k)
        r = np.zeros(264, dtype=np.float32)
        r[0] = 127 * s                                     # row maximum: the scale is exactly s
        r[1:9] = np.array([0.5, -0.5, 1.5, 2.5, 0.49609375, 0.50390625, 0.25, 0.75], dtype=np.float32) * s
        r[9:] = np.linspace(-3, 3, 255, dtype=np.float32) * s
        rows.append(r)
    for dtype in ("f16", "bf16"):
        X = wl.to_bits(np.stack(rows * 3), dtype)
        Xd = to_dev(X, dtype)
        for alpha, theta in [(1.0, 1.0), (1.0, 3.0), (0.0, 1.0), (0.3, 1.0), (1.0, 1e-30), (1.0, 1e30), (0.5, 2.0 ** -21)]:
            want, removed, k_pt, k_cq = orc.remove_kernel(X, dtype, alpha, 8, theta)
            out, counts = cq.remove_kernel(Xd, alpha, 8, theta)
            assert counts.cpu().tolist() == [removed, k_pt, k_cq], (dtype, alpha, theta)
            assert np.array_equal(bits_of(out), want)
            t, c = cq.absmax_rows_cols(Xd)
            assert int(cq.kernel_count_x(Xd, alpha, 8, t, c).item()) == k_cq
    # scale factors outside [2^-40, 2^40]: everything goes through the quotient
    for scale in (1e36, 1e-36, 3e-39):
        B = wl.small_matrix(24, 128, "bf16", 4, scale=scale, outlier_cols=1, outlier_scale=8.0, zero_frac=0.05)
        Bd = to_dev(B, "bf16")
        for alpha in (0.0, 0.15, 1.0):
            want, removed, k_pt, k_cq = orc.remove_kernel(B, "bf16", alpha, 8, 1.0)
            out, counts = cq.remove_kernel(Bd, alpha, 8, 1.0)
            assert counts.cpu().tolist() == [removed, k_pt, k_cq], (scale, alpha)
            assert np.array_equal(bits_of(out), want)


@pytest.mark.parametrize("shape", [(48, 80), (300, 1536), (65, 7), (1, 1)])
def test_case_indicators(cq, shape):
    T, I = shape
    X = wl.small_matrix(T, I, "bf16", 95, dist="laplace", outlier_cols=3, outlier_scale=30.0)
    if I % 2:
        X = X[:, :max(1, I)]
    Xd = to_dev(X, "bf16")
    for alpha in (0.15, 0.75, 1.0):
        r = cq.quantize_act(Xd, alpha, 8)
        got = cq.case_indicators(r).cpu().tolist()
        ref = orc.quantize_act(X, "bf16", alpha, 8, want_deq32=False, want_deq16=False)
        assert tuple(got) == orc.case_indicators(ref.t, ref.c, ref.a, ref.b, 8)


def test_weight_quantizer_equals_alpha_one_activation_path(cq):
    W = wl.small_matrix(64, 1024, "bf16", 61, scale=0.02, outlier_cols=0)
    Wd = to_dev(W, "bf16")
    rw = cq.quantize_weight_per_channel(Wd, 8)
    ra = cq.quantize_act(Wd, 1.0, 8)
    assert torch.equal(rw.codes, ra.codes) and torch.equal(rw.scale, ra.row_scale)


def test_host_buffer_entry_point(cq):
    X = wl.small_matrix(300, 1536, "bf16", 71, outlier_cols=3)
    Xh = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
    for bits in (8, 4):
        buf = cq.HostBuffers(300, 1536, torch.bfloat16, bits)
        r = cq.quantize_act_host(Xh, 0.15, bits, buffers=buf)
        torch.cuda.synchronize()
        parity.check_act(X, "bf16", 0.15, bits, t=r.t.numpy(), c=r.c.numpy(), a=r.row_scale.numpy(),
                         b=r.col_scale.numpy(), codes=r.codes.numpy(),
                         deq=r.deq.view(torch.int16).numpy().view(np.uint16), zero_count=int(r.zero_count.item()))


def test_too_small_workspace_is_rejected_on_the_device(cq):
    Xd = torch.zeros((64, 512), dtype=torch.float16, device="cuda")
    buf = cq.ActBuffers(64, 512, torch.float16, 8)
    buf.workspace = buf.workspace[:1024]
    with pytest.raises(cq.CQError) as e:
        cq.quantize_act(Xd, 0.15, 8, buffers=buf)
    assert e.value.status == 7
