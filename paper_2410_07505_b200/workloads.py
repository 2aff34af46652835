"""Seeded synthetic inputs: activation and weight matrices as raw 16-bit patterns.

This module only *produces inputs*.  It holds none of the quantizer's arithmetic
(no absmax, no scale, no rounding to codes); the same bytes are handed to the CUDA
library and to the CPU checker, so the generator can never influence a comparison.

The matrices stand in for the activations the paper measures on OPT / LLaMA models
(Section 5.1 "Models"; the outlier description in Appendix A: a small share of the
input features carry values at least 20x larger than the rest).  Shapes follow the
named models' layer widths.  All draws come from ``numpy.random.Generator(PCG64(seed))``
in float64/float32, are given their structure (outlier channels, exact zeros,
massive tokens) and are then rounded once, to nearest-even, to fp16 or bf16.

Draw order (part of the recipe, so that every user gets the same bytes):
  1. structure indices that depend on the seed (config "tiny" only),
  2. the matrix in blocks of ``ROW_BLOCK`` consecutive rows; inside a block first the
     values (row-major), then, where the config has one, the Bernoulli zero mask.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

import numpy as np

ROW_BLOCK = 256

F16 = "f16"
BF16 = "bf16"


# --------------------------------------------------------------------------------------
# 16-bit storage formats (format conversion only)
# --------------------------------------------------------------------------------------
def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> IEEE binary16 bit patterns, round-to-nearest-even (numpy's cast)."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == F16:
        return f32_to_f16_bits(x)
    if dtype == BF16:
        return f32_to_bf16_bits(x)
    raise ValueError(f"unknown 16-bit dtype {dtype!r}")


def bits_to_f32(bits: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of fp16 / bf16 bit patterns to float32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == F16:
        return bits.view(np.float16).astype(np.float32)
    if dtype == BF16:
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError(f"unknown 16-bit dtype {dtype!r}")


# --------------------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class ActConfig:
    name: str
    T: int
    I: int
    dtype: str
    dist: str            # "normal" | "student_t3" | "laplace"
    seed: int
    outlier_cols: int    # number of outlier channels
    outlier_kind: str    # "seeded" (indices drawn) | "fixed" (evenly spaced)
    outlier_scale: tuple  # one factor per outlier channel
    zero_frac: float = 0.0
    massive_rows: int = 0       # tokens whose entries in `massive_cols` channels are x1000
    massive_cols: int = 0
    bits: tuple = (8,)
    alphas: tuple = (0.15,)

    @property
    def elements(self) -> int:
        return self.T * self.I


def _fixed_columns(I: int, n: int) -> np.ndarray:
    """n evenly spaced channel indices: ((2k+1) * I) // (2n)."""
    return np.array([((2 * k + 1) * I) // (2 * n) for k in range(n)], dtype=np.int64)


ACT_CONFIGS = {
    # 1 Tiny
    "tiny": ActConfig("tiny", 128, 768, F16, "normal", 0, 4, "seeded", (40.0,) * 4,
                      bits=(8,), alphas=(0.0, 0.15, 0.5, 1.0)),
    # 2 OPT-6.7B-shaped: attention/FC1 input and FC2 input
    "opt6.7b_attn": ActConfig("opt6.7b_attn", 2048, 4096, F16, "normal", 1, 6, "fixed",
                              (20.0, 28.0, 36.0, 44.0, 52.0, 60.0), zero_frac=0.01,
                              bits=(8, 4), alphas=(0.15,)),
    "opt6.7b_fc2": ActConfig("opt6.7b_fc2", 2048, 16384, F16, "normal", 2, 6, "fixed",
                             (20.0, 28.0, 36.0, 44.0, 52.0, 60.0), zero_frac=0.01,
                             bits=(8, 4), alphas=(0.15,)),
    # 3 LLaMA-2-13B-shaped
    "llama13b_attn": ActConfig("llama13b_attn", 4096, 5120, BF16, "student_t3", 3, 0, "fixed", (),
                               massive_rows=2, massive_cols=3, bits=(8, 4), alphas=(0.15, 0.5)),
    "llama13b_mlp": ActConfig("llama13b_mlp", 4096, 13824, BF16, "student_t3", 4, 0, "fixed", (),
                              massive_rows=2, massive_cols=3, bits=(8, 4), alphas=(0.15, 0.5)),
    # 4 LLaMA-70B-shaped
    "llama70b_attn": ActConfig("llama70b_attn", 4096, 8192, BF16, "laplace", 5, 8, "fixed",
                               (50.0,) * 8, bits=(8, 4), alphas=(0.15,)),
    "llama70b_mlp": ActConfig("llama70b_mlp", 4096, 28672, BF16, "laplace", 6, 8, "fixed",
                              (50.0,) * 8, bits=(8, 4), alphas=(0.15,)),
}

HEADLINE = "llama70b_mlp"

# 5 Sweep: 80 layers at 2048 tokens, 4 linear-layer inputs and 3 weight shapes per layer.
SWEEP_LAYERS = 80
SWEEP_TOKENS = 2048
SWEEP_ACT_WIDTHS = (8192, 8192, 8192, 28672)
SWEEP_WEIGHT_SHAPES = ((8192, 8192), (8192, 28672), (28672, 8192))
SWEEP_WEIGHT_STD = 0.02


def _draw_block(rng: np.random.Generator, dist: str, rows: int, cols: int) -> np.ndarray:
    if dist == "normal":
        return rng.standard_normal((rows, cols), dtype=np.float32)
    if dist == "student_t3":
        return rng.standard_t(3.0, size=(rows, cols)).astype(np.float32)
    if dist == "laplace":
        return rng.laplace(0.0, 1.0, size=(rows, cols)).astype(np.float32)
    raise ValueError(dist)


def generate_activation(cfg: ActConfig) -> np.ndarray:
    """Return the T x I matrix of ``cfg`` as uint16 bit patterns of ``cfg.dtype``."""
    rng = np.random.Generator(np.random.PCG64(cfg.seed))
    T, I = cfg.T, cfg.I
    if cfg.outlier_cols:
        if cfg.outlier_kind == "seeded":
            ocols = np.sort(rng.choice(I, size=cfg.outlier_cols, replace=False))
        else:
            ocols = _fixed_columns(I, cfg.outlier_cols)
        oscale = np.asarray(cfg.outlier_scale, dtype=np.float32)
    mrows = mcols = None
    if cfg.massive_rows:
        mrows = [(k * T) // cfg.massive_rows for k in range(cfg.massive_rows)]
        mcols = _fixed_columns(I, cfg.massive_cols)
    out = np.empty((T, I), dtype=np.uint16)
    for r0 in range(0, T, ROW_BLOCK):
        r1 = min(T, r0 + ROW_BLOCK)
        blk = _draw_block(rng, cfg.dist, r1 - r0, I)
        if cfg.zero_frac > 0.0:
            mask = rng.random((r1 - r0, I), dtype=np.float32) < np.float32(cfg.zero_frac)
        if cfg.outlier_cols:
            blk[:, ocols] *= oscale[None, :]
        if mrows is not None:
            for r in mrows:
                if r0 <= r < r1:
                    blk[r - r0, mcols] *= np.float32(1000.0)
        if cfg.zero_frac > 0.0:
            blk[mask] = 0.0
        out[r0:r1] = to_bits(blk, cfg.dtype)
    return out


def activation(name: str) -> tuple[np.ndarray, ActConfig]:
    cfg = ACT_CONFIGS[name]
    return generate_activation(cfg), cfg


def sweep_activation_config(layer: int, k: int, tokens: int = SWEEP_TOKENS) -> ActConfig:
    """k-th linear-layer input (0..3) of `layer` (0..79) of the 80-layer sweep."""
    I = SWEEP_ACT_WIDTHS[k]
    return ActConfig(f"sweep_L{layer}_x{k}", tokens, I, BF16, "laplace", 1000 + 4 * layer + k,
                     8, "fixed", (50.0,) * 8, bits=(8, 4), alphas=(0.15,))


def sweep_weight(layer: int, k: int, shape: tuple | None = None) -> np.ndarray:
    """k-th weight (0..2) of `layer`: bf16 N(0, 0.02^2), stored rows = output channels."""
    R, C = shape if shape is not None else SWEEP_WEIGHT_SHAPES[k]
    rng = np.random.Generator(np.random.PCG64(5000 + 3 * layer + k))
    out = np.empty((R, C), dtype=np.uint16)
    for r0 in range(0, R, ROW_BLOCK):
        r1 = min(R, r0 + ROW_BLOCK)
        blk = rng.standard_normal((r1 - r0, C), dtype=np.float32) * np.float32(SWEEP_WEIGHT_STD)
        out[r0:r1] = f32_to_bf16_bits(blk)
    return out


# --------------------------------------------------------------------------------------
# small / ragged matrices for tests
# --------------------------------------------------------------------------------------
def small_matrix(T: int, I: int, dtype: str, seed: int, dist: str = "normal",
                 outlier_cols: int = 2, outlier_scale: float = 30.0,
                 zero_frac: float = 0.0, scale: float = 1.0) -> np.ndarray:
    """Arbitrary-shape matrix with the same kind of structure as the configs."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if T == 0 or I == 0:
        return np.empty((T, I), dtype=np.uint16)
    blk = _draw_block(rng, dist, T, I) * np.float32(scale)
    n_out = min(outlier_cols, I)
    if n_out:
        cols = np.sort(rng.choice(I, size=n_out, replace=False))
        blk[:, cols] *= np.float32(outlier_scale)
    if zero_frac > 0.0:
        blk[rng.random((T, I), dtype=np.float32) < np.float32(zero_frac)] = 0.0
    return to_bits(blk, dtype)


def iter_sweep(layers: Iterator[int]):
    """Yield (layer, [4 activation configs], [3 weight shapes]) for the given layers."""
    for layer in layers:
        yield layer, [sweep_activation_config(layer, k) for k in range(4)], list(SWEEP_WEIGHT_SHAPES)
