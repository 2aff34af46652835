"""Element-by-element comparison of a result (numpy arrays, wherever they came from) with the
CPU oracle.  TEST INFRASTRUCTURE: used by tests/, the smoke check and nothing else.

The bar (written here once so every caller applies the same one):
  * t, c ........................ bit-exact
  * scale vectors a, b .......... within 2 fp32 ulp (in practice identical: both sides round one
                                  fp64 pow; a last-bit difference of the two pow routines would show here)
  * codes, zero count ........... bit-exact; if (and only if) a scale factor differs by an ulp, code
                                  mismatches are allowed where |x/s| lies within 1e-6 (relative) of a
                                  rounding boundary, at most 1e-6 of the elements
  * dequantized values .......... within 2 fp32 ulp (fp32 output), equal after the final rounding
                                  or one 16-bit ulp apart where the fp32 values differ (16-bit output)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import cq_oracle as orc


def ulp_distance_f32(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    ip = np.ascontiguousarray(p, dtype=np.float32).view(np.int32).astype(np.int64)
    iq = np.ascontiguousarray(q, dtype=np.float32).view(np.int32).astype(np.int64)
    return np.abs(ip - iq)


def unpack_int4(packed: np.ndarray, T: int, I: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8).reshape(T, I // 2)
    lo = (packed & 0xF).astype(np.int8)
    hi = (packed >> 4).astype(np.int8)
    lo = np.where(lo >= 8, lo - 16, lo).astype(np.int8)
    hi = np.where(hi >= 8, hi - 16, hi).astype(np.int8)
    out = np.empty((T, I), dtype=np.int8)
    out[:, 0::2] = lo
    out[:, 1::2] = hi
    return out


@dataclass
class Report:
    scales_identical: bool
    code_mismatches: int
    max_scale_ulp: int
    max_deq_ulp: int
    zero_count: int
    kernel_proportion: float


def check_act(X: np.ndarray, dtype: str, alpha: float, bits: int, *, t=None, c=None, a=None, b=None,
              codes=None, deq=None, deq_is_f32=False, zero_count=None, ref: orc.ActResult | None = None) -> Report:
    """Assert that the given outputs of the activation quantizer match the oracle on X."""
    T, I = X.shape
    if ref is None:
        ref = orc.quantize_act(X, dtype, alpha, bits, want_deq32=True, want_deq16=True)
    if t is not None:
        assert np.array_equal(np.asarray(t).view(np.uint32), ref.t.view(np.uint32)), "row absmax differs"
    if c is not None:
        assert np.array_equal(np.asarray(c).view(np.uint32), ref.c.view(np.uint32)), "column absmax differs"
    max_scale_ulp = 0
    identical = True
    for got, want, name in ((a, ref.a, "row scale"), (b, ref.b, "column scale")):
        if got is None:
            continue
        d = ulp_distance_f32(got, want)
        m = int(d.max()) if d.size else 0
        assert m <= 2, f"{name} off by {m} ulp"
        max_scale_ulp = max(max_scale_ulp, m)
        identical = identical and m == 0
    mismatches = 0
    if codes is not None:
        got = np.asarray(codes)
        got = unpack_int4(got, T, I) if bits == 4 else got.reshape(T, I).view(np.int8)
        diff = got != ref.codes
        mismatches = int(diff.sum())
        if identical:
            assert mismatches == 0, f"{mismatches} codes differ although the scale vectors are identical"
        elif mismatches:
            assert mismatches <= max(1, int(1e-6 * T * I)), f"{mismatches} code mismatches"
            ii, jj = np.nonzero(diff)
            x = orc.decode16(X[ii, jj], dtype).astype(np.float64)
            s = (ref.a[ii] * ref.b[jj]).astype(np.float32).astype(np.float64)
            u = np.abs(x / s)
            boundary = np.floor(u) + 0.5
            assert np.all(np.abs(u - boundary) <= 1e-6 * boundary), "code mismatch away from a rounding boundary"
            assert np.all(np.abs(got[ii, jj].astype(np.int32) - ref.codes[ii, jj].astype(np.int32)) <= 1)
    max_deq_ulp = 0
    if deq is not None:
        got = np.asarray(deq).reshape(T, I)
        if deq_is_f32:
            d = ulp_distance_f32(got, ref.deq32)
            if mismatches:
                d = d[~diff]
            max_deq_ulp = int(d.max()) if d.size else 0
            assert max_deq_ulp <= 2, f"dequantized fp32 value off by {max_deq_ulp} ulp"
            if identical:
                assert max_deq_ulp == 0
        else:
            neq = got.view(np.uint16) != ref.deq16
            if identical:
                assert not neq.any(), f"{int(neq.sum())} dequantized 16-bit values differ"
            else:
                d16 = np.abs(got.view(np.uint16).astype(np.int32) - ref.deq16.astype(np.int32))
                if mismatches:
                    d16 = d16[~diff]
                assert (d16 <= 1).all()
    if zero_count is not None:
        if mismatches == 0:
            assert int(zero_count) == ref.zero_count, f"zero count {int(zero_count)} != {ref.zero_count}"
        else:
            assert abs(int(zero_count) - ref.zero_count) <= mismatches
    return Report(identical, mismatches, max_scale_ulp, max_deq_ulp, ref.zero_count,
                  ref.zero_count / (T * I) if T * I else 0.0)


def check_weight(W: np.ndarray, dtype: str, bits: int, *, scale=None, codes=None, deq=None, deq_is_f32=False,
                 zero_count=None, ref: orc.WeightResult | None = None) -> None:
    """Per-channel weight quantizer: every output bit-exact (no transcendental is involved)."""
    R, Cc = W.shape
    if ref is None:
        ref = orc.quantize_weight_per_channel(W, dtype, bits)
    if scale is not None:
        assert np.array_equal(np.asarray(scale).view(np.uint32), ref.scale.view(np.uint32)), "row scales differ"
    if codes is not None:
        got = np.asarray(codes)
        got = unpack_int4(got, R, Cc) if bits == 4 else got.reshape(R, Cc).view(np.int8)
        assert np.array_equal(got, ref.codes), f"{int((got != ref.codes).sum())} weight codes differ"
    if deq is not None:
        got = np.asarray(deq).reshape(R, Cc)
        if deq_is_f32:
            assert np.array_equal(got.view(np.uint32), ref.deq32.view(np.uint32))
        else:
            assert np.array_equal(got.view(np.uint16), ref.deq16)
    if zero_count is not None:
        assert int(zero_count) == ref.zero_count
