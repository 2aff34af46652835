"""ctypes front end of the CPU oracle (oracle/cq_oracle.c).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It imports nothing from the CUDA
package.  All arrays are numpy, on the host; 16-bit inputs are uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

from . import build as _build

DTYPES = {"f16": 0, "bf16": 1}

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # CQ_ORACLE_LIB lets the mutation tests point the same pins at a deliberately broken build
        path = os.environ.get("CQ_ORACLE_LIB") or _build.build()
        _lib = C.CDLL(path)
        _lib.cqo_kernel_count.restype = C.c_uint64
        _lib.cqo_num_threads.restype = C.c_int
        for name in ("cqo_quantize_act", "cqo_pack_int4", "cqo_quantize_weight_per_channel", "cqo_remove_kernel"):
            getattr(_lib, name).restype = C.c_int
    return _lib


def _p(arr):
    return None if arr is None else arr.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def _check_bits16(X):
    assert X.dtype == np.uint16 and X.ndim == 2 and X.strides[1] == 2
    return X.strides[0] // 2 if (X.shape[0] > 1 and X.shape[1] > 0) else max(X.shape[1], 1)


def num_threads() -> int:
    return int(lib().cqo_num_threads())


def set_num_threads(n: int) -> None:
    """OpenMP threads for later calls (for timing the oracle on one core and on all; results are unaffected)."""
    lib().cqo_set_num_threads(C.c_int(int(n)))


def decode16(bits: np.ndarray, dtype: str) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    lib().cqo_decode16(_p(bits), DTYPES[dtype], _i64(bits.size), _p(out))
    return out


def encode16(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().cqo_encode16(_p(x), DTYPES[dtype], _i64(x.size), _p(out))
    return out


def absmax_rows(X: np.ndarray, dtype: str) -> np.ndarray:
    ld = _check_bits16(X)
    T, I = X.shape
    t = np.empty(T, dtype=np.float32)
    lib().cqo_absmax_rows(_p(X), DTYPES[dtype], _i64(T), _i64(I), _i64(ld), _p(t))
    return t


def absmax_cols(X: np.ndarray, dtype: str) -> np.ndarray:
    ld = _check_bits16(X)
    T, I = X.shape
    c = np.empty(I, dtype=np.float32)
    lib().cqo_absmax_cols(_p(X), DTYPES[dtype], _i64(T), _i64(I), _i64(ld), _p(c))
    return c


def scale_vectors(t, c, alpha: float, bits: int):
    t = np.ascontiguousarray(t, dtype=np.float32)
    c = np.ascontiguousarray(c, dtype=np.float32)
    a = np.empty_like(t)
    b = np.empty_like(c)
    lib().cqo_scale_vectors(_p(t), _p(c), _i64(t.size), _i64(c.size), C.c_double(alpha), C.c_int(bits),
                            _p(a), _p(b))
    return a, b


@dataclass
class ActResult:
    t: np.ndarray
    c: np.ndarray
    a: np.ndarray            # row factor of the scale (carries 1/qmax)
    b: np.ndarray            # column factor of the scale
    codes: np.ndarray | None     # int8 [T, I], one code per element for both bit widths
    deq32: np.ndarray | None     # float32 [T, I]
    deq16: np.ndarray | None     # uint16 [T, I] in X's 16-bit type
    zero_count: int

    def packed_int4(self) -> np.ndarray:
        return pack_int4(self.codes)

    @property
    def kernel_proportion(self) -> float:
        n = self.codes.size if self.codes is not None else self.t.size * self.c.size
        return self.zero_count / n if n else 0.0


def quantize_act(X: np.ndarray, dtype: str, alpha: float, bits: int, *, want_codes=True,
                 want_deq32=True, want_deq16=True, clamp=True) -> ActResult:
    ld = _check_bits16(X)
    T, I = X.shape
    t = np.empty(T, dtype=np.float32)
    c = np.empty(I, dtype=np.float32)
    a = np.empty(T, dtype=np.float32)
    b = np.empty(I, dtype=np.float32)
    codes = np.empty((T, I), dtype=np.int8) if want_codes else None
    deq32 = np.empty((T, I), dtype=np.float32) if want_deq32 else None
    deq16 = np.empty((T, I), dtype=np.uint16) if want_deq16 else None
    zc = C.c_uint64(0)
    rc = lib().cqo_quantize_act(_p(X), DTYPES[dtype], _i64(T), _i64(I), _i64(ld), C.c_double(alpha),
                                C.c_int(bits), _p(t), _p(c), _p(a), _p(b), _p(codes), _p(deq32),
                                _p(deq16), C.byref(zc), C.c_int(1 if clamp else 0))
    if rc != 0:
        raise ValueError("cqo_quantize_act: bad arguments")
    return ActResult(t, c, a, b, codes, deq32, deq16, int(zc.value))


def pack_int4(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    T, I = codes.shape
    out = np.empty((T, I // 2), dtype=np.uint8)
    if lib().cqo_pack_int4(_p(codes), _i64(T), _i64(I), _p(out)) != 0:
        raise ValueError("INT4 packing needs an even number of columns")
    return out


def dequantize(codes: np.ndarray, bits: int, T: int, I: int, a, b, out16_dtype: str | None = None):
    codes = np.ascontiguousarray(codes)
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    out32 = np.empty((T, I), dtype=np.float32)
    out16 = np.empty((T, I), dtype=np.uint16) if out16_dtype else None
    lib().cqo_dequantize(_p(codes), C.c_int(bits), _i64(T), _i64(I), _p(a), _p(b), _p(out32), _p(out16),
                         C.c_int(DTYPES[out16_dtype] if out16_dtype else 0))
    return out32, out16


def kernel_count(codes: np.ndarray, bits: int, T: int, I: int) -> int:
    codes = np.ascontiguousarray(codes)
    return int(lib().cqo_kernel_count(_p(codes), C.c_int(bits), _i64(T), _i64(I)))


@dataclass
class WeightResult:
    scale: np.ndarray
    codes: np.ndarray | None
    deq32: np.ndarray | None
    deq16: np.ndarray | None
    zero_count: int


def quantize_weight_per_channel(W: np.ndarray, dtype: str, bits: int, *, want_codes=True,
                                want_deq32=True, want_deq16=True) -> WeightResult:
    ld = _check_bits16(W)
    R, Cc = W.shape
    scale = np.empty(R, dtype=np.float32)
    codes = np.empty((R, Cc), dtype=np.int8) if want_codes else None
    deq32 = np.empty((R, Cc), dtype=np.float32) if want_deq32 else None
    deq16 = np.empty((R, Cc), dtype=np.uint16) if want_deq16 else None
    zc = C.c_uint64(0)
    rc = lib().cqo_quantize_weight_per_channel(_p(W), DTYPES[dtype], _i64(R), _i64(Cc), _i64(ld),
                                               C.c_int(bits), _p(codes), _p(scale), _p(deq32),
                                               _p(deq16), C.byref(zc))
    if rc != 0:
        raise ValueError("cqo_quantize_weight_per_channel: bad arguments")
    return WeightResult(scale, codes, deq32, deq16, int(zc.value))


def compare_with_ideal(X: np.ndarray, dtype: str, alpha: float, bits: int, res: ActResult,
                       rel: float = 1e-6):
    """(max ulp distance of s_ij from the fp64 ideal, #codes differing from the fp64 ideal,
    #of those farther than `rel` from a rounding boundary)."""
    ld = _check_bits16(X)
    T, I = X.shape
    out = np.zeros(3, dtype=np.int64)
    lib().cqo_compare_with_ideal(_p(X), DTYPES[dtype], _i64(T), _i64(I), _i64(ld), C.c_double(alpha),
                                 C.c_int(bits), _p(res.t), _p(res.c), _p(res.a), _p(res.b),
                                 _p(np.ascontiguousarray(res.codes)), C.c_double(rel), _p(out))
    return int(out[0]), int(out[1]), int(out[2])


def quantize_weight_groupwise(W: np.ndarray, dtype: str, bits: int, group: int) -> WeightResult:
    """Group-wise weight quantization exactly as the paper states it (Section 3): reshape the weight
    matrix to (elements / g) x g, quantize per row (Eq. 2), reshape back."""
    R, Cc = W.shape
    if group <= 0 or Cc % group:
        raise ValueError("the group size must divide the number of columns")
    flat = np.ascontiguousarray(W).reshape(R * Cc // group, group)
    r = quantize_weight_per_channel(flat, dtype, bits)
    return WeightResult(r.scale, r.codes.reshape(R, Cc), r.deq32.reshape(R, Cc), r.deq16.reshape(R, Cc), r.zero_count)


def case_indicators(t, c, a, b, bits: int):
    """(#pairs with c_j >= t_i, #pairs whose CrossQuant zero bound is below the per-token one)."""
    t = np.ascontiguousarray(t, dtype=np.float32)
    c = np.ascontiguousarray(c, dtype=np.float32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    out = np.zeros(2, dtype=np.uint64)
    lib().cqo_case_indicators(_p(t), _p(c), _p(a), _p(b), _i64(t.size), _i64(c.size), C.c_int(bits), _p(out))
    return int(out[0]), int(out[1])


def remove_kernel(X: np.ndarray, dtype: str, alpha: float, bits: int, bound_scale: float = 1.0):
    """Remove-Kernel operator: (matrix with the kernel elements set to +0 and the rest untouched,
    #removed, |K(Q)| per-token, |K(CQ)| for alpha)."""
    ld = _check_bits16(X)
    T, I = X.shape
    out = np.empty((T, I), dtype=np.uint16)
    counts = np.zeros(3, dtype=np.uint64)
    rc = lib().cqo_remove_kernel(_p(X), DTYPES[dtype], _i64(T), _i64(I), _i64(ld), C.c_double(alpha), C.c_int(bits),
                                 C.c_float(bound_scale), _p(out), _p(counts))
    if rc != 0:
        raise ValueError("cqo_remove_kernel: bad arguments")
    return out, int(counts[0]), int(counts[1]), int(counts[2])
