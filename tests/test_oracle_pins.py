"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here calls the CUDA path.  Each pin is independent of the oracle's own code:
numpy / torch format casts, exact integer or 50-digit decimal arithmetic, closed forms,
invariants of the CrossQuant equation, and the special cases the paper states
(alpha = 1 is per-token quantization, Table 1 caption; by symmetry alpha = 0 is
per-column quantization).
"""
from __future__ import annotations

import itertools
import math
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest

import codecs16
from oracle import cq_oracle as orc
from paper_2410_07505_b200 import workloads as wl

QMAX = {8: 127, 4: 7}


def dec(bits, dtype):
    """Decoder that is not the oracle's: numpy (fp16) / widened bit pattern (bf16), tests/codecs16.py."""
    return codecs16.bits_to_f32(bits, dtype)


def rand_matrix(T, I, dtype, seed, **kw):
    return wl.small_matrix(T, I, dtype, seed, **kw)


# ------------------------------------------------------------------ 16-bit formats ---
def test_decode_f16_all_patterns_matches_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.decode16(bits, "f16")
    ref = bits.view(np.float16).astype(np.float32)
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite].view(np.uint32), ref[finite].view(np.uint32))
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))


def test_decode_bf16_all_patterns_matches_torch():
    import torch
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.decode16(bits, "bf16")
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok].view(np.uint32), ref[ok].view(np.uint32))
    assert np.array_equal(np.isnan(got), np.isnan(ref))


def _encode_probe_values():
    rng = np.random.Generator(np.random.PCG64(11))
    parts = [
        rng.standard_normal(200000).astype(np.float32),
        (rng.standard_normal(100000) * 1e-6).astype(np.float32),       # fp16 subnormal range
        (rng.standard_normal(100000) * 3e4).astype(np.float32),        # near fp16 overflow
        np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e30, -1e30, 2.0 ** -14, 2.0 ** -24,
                  2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14 - 2.0 ** -25, 2.0 ** -14 - 2.0 ** -26],
                 dtype=np.float32),
    ]
    # exact halfway cases between adjacent fp16 values and between adjacent bf16 values
    h = np.arange(0x0001, 0x7BFF, 37, dtype=np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + np.uint16(1)).view(np.float16).astype(np.float64)
    parts.append(((lo + hi) / 2).astype(np.float32))
    b = np.arange(0x0080, 0x7F00, 53, dtype=np.uint32)
    parts.append(((b << 16) | 0x8000).astype(np.uint32).view(np.float32))
    v = np.concatenate(parts)
    return np.concatenate([v, -v])


def test_encode_f16_matches_numpy_cast():
    v = _encode_probe_values()
    with np.errstate(over="ignore"):
        ref = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(orc.encode16(v, "f16"), ref)


def test_encode_bf16_matches_torch_cast():
    import torch
    v = _encode_probe_values()
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.encode16(v, "bf16"), ref)


# ------------------------------------------------------------------ absmax vectors ---
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_absmax_is_the_plain_definition(dtype):
    X = rand_matrix(37, 53, dtype, 5)
    x = dec(X, dtype)
    t = orc.absmax_rows(X, dtype)
    c = orc.absmax_cols(X, dtype)
    # brute force with exact rationals, element by element
    for i in range(X.shape[0]):
        assert Fraction(float(t[i])) == max(abs(Fraction(float(v))) for v in x[i])
    for j in range(X.shape[1]):
        assert Fraction(float(c[j])) == max(abs(Fraction(float(v))) for v in x[:, j])


def test_absmax_respects_leading_dimension():
    big = rand_matrix(16, 40, "bf16", 6)
    view = big[:, 3:29]
    assert np.array_equal(orc.absmax_rows(view, "bf16"), np.abs(dec(view, "bf16")).max(axis=1))
    assert np.array_equal(orc.absmax_cols(view, "bf16"), np.abs(dec(view, "bf16")).max(axis=0))


# ------------------------------------------------------------------ special cases ----
@pytest.mark.parametrize("dtype,bits", [("f16", 8), ("bf16", 8), ("f16", 4), ("bf16", 4)])
def test_alpha_one_is_per_token_quantization(dtype, bits):
    """Eq. 1 written with numpy float32 ops (IEEE division, rint = ties-to-even)."""
    X = rand_matrix(64, 96, dtype, 21, outlier_cols=3)
    x = dec(X, dtype)
    t = np.abs(x).max(axis=1)
    delta = (t / np.float32(QMAX[bits])).astype(np.float32)[:, None]
    q = np.rint((x / delta).astype(np.float32)).astype(np.int32)
    xhat = (q.astype(np.float32) * delta).astype(np.float32)
    r = orc.quantize_act(X, dtype, 1.0, bits)
    assert np.array_equal(r.codes.astype(np.int32), q)
    assert np.array_equal(r.deq32.view(np.uint32), xhat.view(np.uint32))
    assert r.zero_count == int((q == 0).sum())
    assert np.all(r.b == 1.0)


@pytest.mark.parametrize("dtype,bits", [("f16", 8), ("bf16", 4)])
def test_alpha_zero_is_per_column_quantization(dtype, bits):
    X = rand_matrix(64, 96, dtype, 22, outlier_cols=3)
    x = dec(X, dtype)
    c = np.abs(x).max(axis=0)
    delta = (c / np.float32(QMAX[bits])).astype(np.float32)[None, :]
    q = np.rint((x / delta).astype(np.float32)).astype(np.int32)
    r = orc.quantize_act(X, dtype, 0.0, bits)
    assert np.array_equal(r.codes.astype(np.int32), q)
    assert np.array_equal(r.deq32.view(np.uint32), (q.astype(np.float32) * delta).astype(np.float32).view(np.uint32))
    assert np.all(r.a == 1.0)


@pytest.mark.parametrize("bits", [8, 4])
def test_weight_quantizer_equals_per_token_on_the_same_matrix(bits):
    """Eq. 2 on stored rows is Eq. 1 on the same matrix (two separately written loops)."""
    W = rand_matrix(48, 200, "bf16", 23, scale=0.02, outlier_cols=0)
    rw = orc.quantize_weight_per_channel(W, "bf16", bits)
    ra = orc.quantize_act(W, "bf16", 1.0, bits)
    assert np.array_equal(rw.codes, ra.codes)
    assert np.array_equal(rw.scale, ra.a)
    assert np.array_equal(rw.deq32.view(np.uint32), ra.deq32.view(np.uint32))
    assert np.array_equal(rw.deq16, ra.deq16)
    assert rw.zero_count == ra.zero_count


# ------------------------------------------------------------------ worked example ---
def test_hand_worked_2x2_example():
    """X = [[1, 3], [-4, 8]], alpha = 1/2: t = (3, 8), c = (4, 8) and
    u_ij = x_ij * qmax / sqrt(t_i c_j):
      INT8: 127/sqrt(12) = 36.66, 381/sqrt(24) = 77.77, -508/sqrt(32) = -89.80, 1016/sqrt(64) = 127
      INT4:   7/sqrt(12) =  2.02,  21/sqrt(24) =  4.29,  -28/sqrt(32) =  -4.95,   56/sqrt(64) = 7
    none of them near a rounding boundary."""
    X = codecs16.to_bits(np.array([[1, 3], [-4, 8]], dtype=np.float32), "f16")
    r8 = orc.quantize_act(X, "f16", 0.5, 8)
    assert r8.t.tolist() == [3.0, 8.0] and r8.c.tolist() == [4.0, 8.0]
    assert r8.codes.tolist() == [[37, 78], [-90, 127]]
    assert r8.zero_count == 0
    r4 = orc.quantize_act(X, "f16", 0.5, 4)
    assert r4.codes.tolist() == [[2, 4], [-5, 7]]
    # dequantized values: q * sqrt(t c) / qmax
    want = np.array([[37 * math.sqrt(12) / 127, 78 * math.sqrt(24) / 127],
                     [-90 * math.sqrt(32) / 127, 8.0]])
    assert np.allclose(r8.deq32, want, rtol=4e-7, atol=0)


def test_ties_round_to_even_as_in_the_listing():
    """Appendix B.1's listing rounds with torch.round (ties to even).  With alpha = 1 and a row
    maximum of 127 the step is exactly 1, so u = x and the ties are exact."""
    row = np.array([[127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 126.5, -125.5]], dtype=np.float32)
    r = orc.quantize_act(codecs16.to_bits(row, "f16"), "f16", 1.0, 8)
    assert r.codes.tolist() == [[127, 0, 2, 2, 0, -2, -2, 4, 126, -126]]
    assert r.zero_count == 2            # |u| = 1/2 exactly lands in the kernel under this reading


def test_kernel_example_small_values_fall_to_zero_only_per_token():
    """One outlier channel: per-token sends the small entries of every row to zero, the
    cross scale keeps them (the situation of the paper's Section 4.2 discussion)."""
    x = np.full((4, 8), 0.3, dtype=np.float32)
    x[:, 5] = 100.0
    X = codecs16.to_bits(x, "f16")
    per_token = orc.quantize_act(X, "f16", 1.0, 8)
    cross = orc.quantize_act(X, "f16", 0.15, 8)
    assert per_token.zero_count == 4 * 7        # 0.3 * 127 / 100 = 0.381 < 1/2
    assert cross.zero_count == 0
    assert np.all(cross.codes[:, 5] == 127)


# ------------------------------------------------------------------ invariants -------
ALPHAS = [0.0, 0.15, 0.45, 0.5, 0.75, 1.0]


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("bits", [8, 4])
def test_codes_stay_in_range_without_the_clamp(dtype, bits):
    for alpha in ALPHAS:
        X = rand_matrix(96, 160, dtype, 31 + int(alpha * 100), outlier_cols=4, outlier_scale=50.0)
        r = orc.quantize_act(X, dtype, alpha, bits, clamp=False)
        assert r.codes.min() >= -QMAX[bits] and r.codes.max() <= QMAX[bits]
        rc = orc.quantize_act(X, dtype, alpha, bits, clamp=True)
        assert np.array_equal(r.codes, rc.codes)


@pytest.mark.parametrize("bits", [8, 4])
def test_global_absmax_element_gets_qmax(bits):
    X = rand_matrix(40, 72, "f16", 41)
    x = dec(X, "f16")
    i, j = np.unravel_index(np.argmax(np.abs(x)), x.shape)
    for alpha in ALPHAS:
        r = orc.quantize_act(X, "f16", alpha, bits)
        assert r.codes[i, j] == int(np.sign(x[i, j])) * QMAX[bits]
    # alpha = 1: every non-zero row holds +-qmax; alpha = 0: every non-zero column does
    r1 = orc.quantize_act(X, "f16", 1.0, bits)
    assert np.all(np.abs(r1.codes.astype(np.int32)).max(axis=1) == QMAX[bits])
    r0 = orc.quantize_act(X, "f16", 0.0, bits)
    assert np.all(np.abs(r0.codes.astype(np.int32)).max(axis=0) == QMAX[bits])


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("bits", [8, 4])
def test_dequantization_error_is_at_most_half_a_step(dtype, bits):
    for alpha in ALPHAS:
        X = rand_matrix(80, 120, dtype, 51, dist="student_t3", outlier_cols=3)
        x = dec(X, dtype).astype(np.float64)
        r = orc.quantize_act(X, dtype, alpha, bits)
        s = (r.a[:, None] * r.b[None, :]).astype(np.float32).astype(np.float64)
        err = np.abs(x - r.codes.astype(np.float64) * s)
        slack = 4.0 * 2.0 ** -24 * np.abs(x)
        assert np.all(err <= s / 2 + slack)
        # and the stored fp32 dequantized value is q*s rounded once
        assert np.all(np.abs(r.deq32.astype(np.float64) - r.codes * s) <= 2.0 ** -24 * np.abs(r.codes * s))


@pytest.mark.parametrize("alpha", ALPHAS)
def test_all_zero_row_and_column_give_zeros(alpha):
    X = rand_matrix(20, 24, "bf16", 61, outlier_cols=0)
    X[7, :] = 0
    X[:, 11] = 0x8000          # negative zeros
    r = orc.quantize_act(X, "bf16", alpha, 8)
    assert np.all(r.codes[7, :] == 0) and np.all(r.codes[:, 11] == 0)
    assert np.all(r.deq32[7, :] == 0) and np.all(r.deq32[:, 11] == 0)
    assert np.all(np.isfinite(r.deq32))
    assert r.t[7] == 0 and r.c[11] == 0
    # the remaining entries are what the matrix without that row and column gives
    keep_r = [i for i in range(20) if i != 7]
    keep_c = [j for j in range(24) if j != 11]
    sub = np.ascontiguousarray(X[np.ix_(keep_r, keep_c)])
    rs = orc.quantize_act(sub, "bf16", alpha, 8)
    assert np.array_equal(r.codes[np.ix_(keep_r, keep_c)], rs.codes)
    assert r.zero_count == rs.zero_count + 20 + 24 - 1


def test_all_zero_matrix():
    X = np.zeros((5, 6), dtype=np.uint16)
    for alpha in ALPHAS:
        r = orc.quantize_act(X, "f16", alpha, 4)
        assert r.zero_count == 30 and not r.codes.any() and not r.deq32.any()


@pytest.mark.parametrize("alpha", [0.15, 0.5, 1.0])
def test_sign_symmetry(alpha):
    X = rand_matrix(33, 47, "f16", 71)
    r = orc.quantize_act(X, "f16", alpha, 8)
    rn = orc.quantize_act(X ^ np.uint16(0x8000), "f16", alpha, 8)
    assert np.array_equal(rn.codes, -r.codes)
    assert np.array_equal(rn.t, r.t) and np.array_equal(rn.c, r.c)
    assert rn.zero_count == r.zero_count
    assert np.array_equal(rn.deq32, -r.deq32)


@pytest.mark.parametrize("alpha", [0.0, 0.15, 0.5])
def test_row_and_column_permutation_equivariance(alpha):
    X = rand_matrix(29, 38, "bf16", 81)
    rng = np.random.Generator(np.random.PCG64(82))
    pr, pc = rng.permutation(29), rng.permutation(38)
    r = orc.quantize_act(X, "bf16", alpha, 8)
    rp = orc.quantize_act(np.ascontiguousarray(X[np.ix_(pr, pc)]), "bf16", alpha, 8)
    assert np.array_equal(rp.codes, r.codes[np.ix_(pr, pc)])
    assert np.array_equal(rp.t, r.t[pr]) and np.array_equal(rp.c, r.c[pc])
    assert np.array_equal(rp.deq16, r.deq16[np.ix_(pr, pc)])


def test_power_of_two_rescaling_is_exact():
    """t, c, s scale by 2^k exactly when alpha's powers stay exact: alpha = 0.5, k even."""
    X = rand_matrix(16, 16, "bf16", 91, outlier_cols=1)
    x = dec(X, "bf16")
    X4 = codecs16.to_bits(x * np.float32(16.0), "bf16")
    r, r4 = orc.quantize_act(X, "bf16", 0.5, 8), orc.quantize_act(X4, "bf16", 0.5, 8)
    assert np.array_equal(r4.t, r.t * 16) and np.array_equal(r4.c, r.c * 16)
    # codes may differ only through the last-bit rounding of pow; they must agree almost everywhere
    assert (r4.codes != r.codes).mean() < 1e-3


# ------------------------------------------------------------------ exact arithmetic -
def _exact_code_alpha_half(kx, kt, kc, qmax):
    """round-half-even(x*qmax/sqrt(t*c)) for x = kx/4, t = kt/4, c = kc/4 in integers.
    Returns (code, distance_flag) where distance_flag is True if u is within 1e-6 (relative)
    of a rounding boundary, including exact ties."""
    if kt == 0 or kc == 0:
        return 0, False
    n = abs(kx) * qmax                  # |u| = n / sqrt(kt*kc)
    d = kt * kc
    # largest q with (2q-1)^2 * d <= (2n)^2  ->  q = floor(u + 1/2)
    q = (math.isqrt((4 * n * n) // d) + 1) // 2
    while (2 * q + 1) ** 2 * d <= 4 * n * n:
        q += 1
    while q > 0 and (2 * q - 1) ** 2 * d > 4 * n * n:
        q -= 1
    tie = q > 0 and (2 * q - 1) ** 2 * d == 4 * n * n
    if tie and q % 2 == 1:              # u = q - 1/2 exactly; half-even picks the even neighbour
        q -= 1
    u = n / math.sqrt(d)
    near = any(abs(u - bnd) <= 2e-6 * bnd for bnd in (q - 0.5, q + 0.5) if bnd > 0)
    return (q if kx >= 0 else -q), (near or tie)


@pytest.mark.parametrize("bits", [8, 4])
def test_alpha_half_against_exact_integer_arithmetic_all_2x2(bits):
    alphabet = [-12, -7, -4, -3, -1, 0, 1, 2, 3, 5, 8, 12]       # entries k/4, exact in fp16
    qmax = QMAX[bits]
    checked = flagged = 0
    for ks in itertools.product(alphabet, repeat=4):
        k = np.array(ks, dtype=np.int64).reshape(2, 2)
        X = codecs16.to_bits((k / 4.0).astype(np.float32), "f16")
        r = orc.quantize_act(X, "f16", 0.5, bits, want_deq32=False, want_deq16=False)
        kt = np.abs(k).max(axis=1)
        kc = np.abs(k).max(axis=0)
        for i in range(2):
            for j in range(2):
                want, near = _exact_code_alpha_half(int(k[i, j]), int(kt[i]), int(kc[j]), qmax)
                if near:
                    flagged += 1
                    assert abs(int(r.codes[i, j]) - want) <= 1
                else:
                    checked += 1
                    assert int(r.codes[i, j]) == want, (ks, i, j)
    assert checked > 50000 and flagged < checked // 10


@pytest.mark.parametrize("bits", [8, 4])
def test_alpha_half_against_exact_integer_arithmetic_random_2x3(bits):
    rng = np.random.Generator(np.random.PCG64(101))
    qmax = QMAX[bits]
    for _ in range(3000):
        k = rng.integers(-12, 13, size=(2, 3))
        X = codecs16.to_bits((k / 4.0).astype(np.float32), "bf16")
        r = orc.quantize_act(X, "bf16", 0.5, bits, want_deq32=False, want_deq16=False)
        kt, kc = np.abs(k).max(axis=1), np.abs(k).max(axis=0)
        for i in range(2):
            for j in range(3):
                want, near = _exact_code_alpha_half(int(k[i, j]), int(kt[i]), int(kc[j]), qmax)
                if not near:
                    assert int(r.codes[i, j]) == want


@pytest.mark.parametrize("alpha", [0.15, 0.45, 0.55, 0.75, 0.9])
@pytest.mark.parametrize("bits", [8, 4])
def test_general_alpha_against_50_digit_decimal(alpha, bits):
    """The CrossQuant equation evaluated with 50 significant digits on small random matrices."""
    getcontext().prec = 50
    qmax = QMAX[bits]
    d_alpha = Decimal(alpha)             # the double, exactly
    near = total = 0
    for seed in range(6):
        X = rand_matrix(9, 11, "f16" if seed % 2 else "bf16", 200 + seed, outlier_cols=1)
        dtype = "f16" if seed % 2 else "bf16"
        x = dec(X, dtype)
        r = orc.quantize_act(X, dtype, alpha, bits)
        t = [max(abs(Decimal(float(v))) for v in row) for row in x]
        c = [max(abs(Decimal(float(v))) for v in x[:, j]) for j in range(x.shape[1])]
        for i in range(x.shape[0]):
            for j in range(x.shape[1]):
                s = (t[i] ** d_alpha) * (c[j] ** (Decimal(1) - d_alpha)) / qmax
                u = Decimal(float(x[i, j])) / s
                au = abs(u)
                fl = au.to_integral_value(rounding="ROUND_FLOOR")
                boundary = fl + Decimal("0.5")
                want = int(u.to_integral_value(rounding="ROUND_HALF_EVEN"))
                total += 1
                if abs(au - boundary) <= Decimal("1e-6") * boundary:
                    near += 1
                    continue
                assert int(r.codes[i, j]) == want
                # scale within 2 fp32 ulp of the exact one
                s32 = np.float32(r.a[i]) * np.float32(r.b[j])
                assert abs(Decimal(float(s32)) - s) <= 2 * Decimal(float(np.spacing(s32)))
    assert near <= total // 100


@pytest.mark.parametrize("alpha", [0.15, 0.5, 1.0])
def test_kernel_count_matches_the_zero_bound(alpha):
    """Definition 1: code == 0  <=>  |x| < B = s/2 (differences only at exact ties)."""
    X = rand_matrix(128, 192, "f16", 301, outlier_cols=4, outlier_scale=40.0, zero_frac=0.01)
    x = dec(X, "f16").astype(np.float64)
    r = orc.quantize_act(X, "f16", alpha, 8)
    s = (r.a[:, None] * r.b[None, :]).astype(np.float32).astype(np.float64)
    below = np.abs(x) < 0.5 * s
    tie = np.abs(x) == 0.5 * s
    assert int(below.sum()) <= r.zero_count <= int(below.sum() + tie.sum())
    assert r.zero_count == int((r.codes == 0).sum())
    assert r.zero_count == orc.kernel_count(r.codes, 8, *X.shape)


def test_scale_within_two_ulp_of_fp64_evaluation():
    X = rand_matrix(64, 64, "bf16", 401, dist="laplace", outlier_cols=3, outlier_scale=50.0)
    for alpha in [0.15, 0.45, 0.75]:
        for bits in (8, 4):
            r = orc.quantize_act(X, "bf16", alpha, bits)
            ideal = (r.t.astype(np.float64)[:, None] ** alpha) * (r.c.astype(np.float64)[None, :] ** (1 - alpha)) / QMAX[bits]
            s = (r.a[:, None] * r.b[None, :]).astype(np.float32)
            ulps = np.abs(s.view(np.int32).astype(np.int64) - ideal.astype(np.float32).view(np.int32).astype(np.int64))
            assert ulps.max() <= 2
            max_ulp, differ, far = orc.compare_with_ideal(X, "bf16", alpha, bits, r)
            assert max_ulp <= 2 and far == 0 and differ <= 1e-5 * X.size + 1


# ------------------------------------------------------------------ storage ----------
def test_int4_packing_layout():
    codes = np.array([[1, -1, 7, -7], [0, 3, -8 + 1, 2]], dtype=np.int8)
    packed = orc.pack_int4(codes)
    assert packed.tolist() == [[0xF1, 0x97], [0x30, 0x29]]
    assert orc.kernel_count(packed, 4, 2, 4) == 1
    a = np.array([0.5, 2.0], dtype=np.float32)
    b = np.array([1.0, 2.0, 4.0, 0.25], dtype=np.float32)
    out32, _ = orc.dequantize(packed, 4, 2, 4, a, b)
    assert out32.tolist() == [[0.5, -1.0, 14.0, -0.875], [0.0, 12.0, -56.0, 1.0]]


def test_dequantize_reproduces_the_fused_output():
    X = rand_matrix(30, 44, "bf16", 501)
    for bits in (8, 4):
        r = orc.quantize_act(X, "bf16", 0.15, bits)
        stored = r.codes if bits == 8 else r.packed_int4()
        out32, out16 = orc.dequantize(stored, bits, 30, 44, r.a, r.b, "bf16")
        assert np.array_equal(out32.view(np.uint32), r.deq32.view(np.uint32))
        assert np.array_equal(out16, r.deq16)
        assert np.array_equal(r.deq16, codecs16.f32_to_bf16_bits(r.deq32))


def test_deq16_is_deq32_rounded_once_fp16():
    X = rand_matrix(30, 44, "f16", 502)
    r = orc.quantize_act(X, "f16", 0.15, 8)
    assert np.array_equal(r.deq16, codecs16.f32_to_f16_bits(r.deq32))


def test_bad_arguments_are_rejected():
    X = rand_matrix(4, 4, "f16", 1)
    for alpha, bits in [(-0.1, 8), (1.5, 8), (float("nan"), 8), (0.5, 3), (0.5, 16)]:
        with pytest.raises(ValueError):
            orc.quantize_act(X, "f16", alpha, bits)


def test_trend_crossquant_kernel_smaller_than_per_token_on_outlier_data():
    """Reported, and true for this seeded matrix; the paper's Case II shows it is not a theorem."""
    X, cfg = wl.activation("tiny")
    cross = orc.quantize_act(X, cfg.dtype, 0.15, 8).kernel_proportion
    per_token = orc.quantize_act(X, cfg.dtype, 1.0, 8).kernel_proportion
    assert cross < per_token


# ------------------------------------------------------------------ group-wise weights
def test_groupwise_is_per_row_quantization_of_the_reshaped_matrix():
    """Section 3: reshape to (elements / g) x g, then Eq. 2.  Checked against numpy fp32 ops on the groups."""
    W = rand_matrix(6, 256, "bf16", 601, scale=0.02, outlier_cols=1, outlier_scale=10.0)
    w = dec(W, "bf16")
    for g, bits in [(128, 4), (64, 8), (256, 4)]:
        r = orc.quantize_weight_groupwise(W, "bf16", bits, g)
        grp = w.reshape(-1, g)
        d = (np.abs(grp).max(axis=1) / np.float32(QMAX[bits])).astype(np.float32)[:, None]
        q = np.rint((grp / d).astype(np.float32)).astype(np.int32)
        assert np.array_equal(r.codes.reshape(-1, g).astype(np.int32), q)
        assert np.array_equal(r.scale, d[:, 0])
        assert r.scale.shape == (6 * 256 // g,)
    full = orc.quantize_weight_groupwise(W, "bf16", 8, 256)
    per_channel = orc.quantize_weight_per_channel(W, "bf16", 8)
    assert np.array_equal(full.codes, per_channel.codes) and np.array_equal(full.scale, per_channel.scale)
    with pytest.raises(ValueError):
        orc.quantize_weight_groupwise(W, "bf16", 4, 100)


# ------------------------------------------------------------------ Table 1 indicators
def test_case_indicators_brute_force_and_relations():
    """Cases I / II of Section 4.2: c_j >= t_i  <=>  the CrossQuant bound is not below the per-token
    bound (alpha < 1, t_i > 0, in real arithmetic); alpha = 1 makes the two bounds equal."""
    X = rand_matrix(48, 80, "bf16", 701, dist="laplace", outlier_cols=3, outlier_scale=30.0)
    for alpha in (0.15, 0.45, 0.75):
        r = orc.quantize_act(X, "bf16", alpha, 8, want_deq32=False, want_deq16=False)
        n2, nb = orc.case_indicators(r.t, r.c, r.a, r.b, 8)
        t64, c64 = r.t.astype(np.float64), r.c.astype(np.float64)
        case2 = c64[None, :] >= t64[:, None]
        assert n2 == int(case2.sum())
        # exact evaluation of t^alpha c^(1-alpha) < t; pairs within 1e-6 of equality may go either way
        ratio = (c64[None, :] / t64[:, None]) ** (1 - alpha)
        sure = np.abs(ratio - 1) > 1e-6
        assert int(((ratio < 1) & sure).sum()) <= nb <= int(((ratio < 1) | ~sure).sum())
        assert abs((n2 + nb) - X.size) <= int((~sure).sum())
    r1 = orc.quantize_act(X, "bf16", 1.0, 8, want_deq32=False, want_deq16=False)
    assert orc.case_indicators(r1.t, r1.c, r1.a, r1.b, 8)[1] == 0
    # hand example: t = (2, 8), c = (4, 8): pairs with c >= t: (0,0), (0,1), (1,1)
    Xh = codecs16.to_bits(np.array([[1, 2], [-4, 8]], dtype=np.float32), "f16")
    rh = orc.quantize_act(Xh, "f16", 0.5, 8)
    assert orc.case_indicators(rh.t, rh.c, rh.a, rh.b, 8) == (3, 1)


# ------------------------------------------------------------------ Remove Kernel
def test_remove_kernel_zeroes_exactly_the_kernel_and_touches_nothing_else():
    X = rand_matrix(96, 160, "f16", 801, outlier_cols=4, outlier_scale=40.0, zero_frac=0.01)
    x = dec(X, "f16")
    for alpha in (0.15, 1.0):
        q = orc.quantize_act(X, "f16", alpha, 8, want_deq32=False, want_deq16=False)
        out, removed, k_pt, k_cq = orc.remove_kernel(X, "f16", alpha, 8)
        want = np.where(q.codes == 0, np.uint16(0), X)
        assert np.array_equal(out, want)
        assert removed == k_cq == q.zero_count
        assert k_pt == orc.quantize_act(X, "f16", 1.0, 8, want_deq32=False, want_deq16=False).zero_count
    # alpha = 1 against numpy fp32 ops: kernel of Eq. 1 is |x / Delta| <= 1/2
    t = np.abs(x).max(axis=1)
    u = (x / (t / np.float32(127)).astype(np.float32)[:, None]).astype(np.float32)
    out, removed, k_pt, _ = orc.remove_kernel(X, "f16", 1.0, 8)
    assert removed == k_pt == int((np.abs(u) <= 0.5).sum())
    assert np.array_equal(out, np.where(np.abs(u) <= 0.5, np.uint16(0), X))


def test_remove_kernel_hand_example_with_elements_exactly_on_the_bound():
    """Per-token scale 1 (row maximum 127): |x / s| is |x| itself, so the bound theta / 2 can be hit exactly.
    An element ON the bound is removed (for theta = 1 it is the tie that rounds half to even, to code 0)."""
    row = np.array([[127, 0.5, -0.5, 0.75, 1.5, -1.5, 1.25, 2.0]], dtype=np.float32)
    X = codecs16.to_bits(row, "f16")
    out, removed, k_pt, k_cq = orc.remove_kernel(X, "f16", 1.0, 8, 1.0)            # bound 1/2
    assert (removed, k_pt, k_cq) == (2, 2, 2)
    assert np.array_equal(codecs16.bits_to_f32(out, "f16"), [[127, 0, 0, 0.75, 1.5, -1.5, 1.25, 2.0]])
    out, removed, k_pt, k_cq = orc.remove_kernel(X, "f16", 1.0, 8, 3.0)            # bound 3/2: +-1.5 go, 2.0 stays
    assert (removed, k_pt, k_cq) == (6, 2, 2)
    assert np.array_equal(codecs16.bits_to_f32(out, "f16"), [[127, 0, 0, 0, 0, 0, 0, 2.0]])
    out, removed, _, _ = orc.remove_kernel(X, "f16", 1.0, 8, 2.5)                  # bound 5/4: 1.25 is on it
    assert removed == 4 and np.array_equal(codecs16.bits_to_f32(out, "f16"), [[127, 0, 0, 0, 1.5, -1.5, 0, 2.0]])


def test_remove_kernel_bound_scale_sweeps_the_proportion():
    X = rand_matrix(64, 128, "bf16", 802, outlier_cols=3, outlier_scale=30.0)
    x = np.abs(dec(X, "bf16"))
    prev = -1
    for theta in (0.0, 0.5, 1.0, 2.0, 8.0, 1e9):
        out, removed, k_pt, k_cq = orc.remove_kernel(X, "bf16", 0.15, 8, theta)
        assert removed >= prev
        prev = removed
        assert int((out == 0).sum()) >= removed            # removed elements are +0; kept ones are bit-identical
        kept = out != 0
        assert np.array_equal(out[kept], X[kept])
        assert k_cq == orc.remove_kernel(X, "bf16", 0.15, 8, 1.0)[1]
    assert orc.remove_kernel(X, "bf16", 0.15, 8, 0.0)[1] == int((x == 0).sum())
    assert orc.remove_kernel(X, "bf16", 0.15, 8, 1e9)[1] == X.size
    with pytest.raises(ValueError):
        orc.remove_kernel(X, "bf16", 0.15, 8, -1.0)
