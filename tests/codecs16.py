"""fp16 / bf16 <-> fp32 conversions for the pins, written here so that what pins the oracle's own codecs lives with
the tests and is neither the oracle's code nor the product package's.

fp16 goes through numpy's IEEE binary16 type; bf16 is the top half of the binary32 pattern: widening appends 16 zero
bits, narrowing rounds to nearest with ties to the even 16-bit pattern (finite inputs).
"""
from __future__ import annotations

import numpy as np


def bits_to_f32(bits: np.ndarray, dtype: str) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "f16":
        return bits.view(np.float16).astype(np.float32)
    if dtype == "bf16":
        return (bits.astype(np.uint32) * np.uint32(65536)).view(np.float32)
    raise ValueError(dtype)


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    low, high = u & 0xFFFF, u >> 16
    up = (low > 0x8000) | ((low == 0x8000) & ((high & 1) == 1))      # above the midpoint, or on it with an odd pattern
    return (high + up).astype(np.uint16)


def to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f16":
        return f32_to_f16_bits(x)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)
