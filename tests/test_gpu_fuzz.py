"""Seeded random shapes, value structures, exponents and bit widths through every quantizer entry point, each
case against the oracle: inputs with few mantissa bits (rounding ties everywhere), heavy tails with exact
zeros, outlier rows and channels, pure powers of two, zero rows and columns."""
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


def draw_case(rng):
    dtype = ("f16", "bf16")[rng.integers(2)]
    T = int(rng.choice([rng.integers(1, 40), rng.integers(1, 200), rng.integers(200, 900)]))
    I = int(rng.choice([8, 16, 64, 264, 776, 1024, 2056, 4104, 4096, 8192, int(rng.integers(1, 3000))]))
    bits = (8, 4)[rng.integers(2)]
    if bits == 4 and I % 2:
        I += 1
    alpha = float(rng.choice([0.0, 0.15, 0.5, 0.75, 1.0, rng.random()]))
    mode = int(rng.integers(4))
    if mode == 0:        # few mantissa bits: ties everywhere
        x = rng.integers(-64, 65, size=(T, I)).astype(np.float32) * np.float32(2.0 ** rng.integers(-12, 6))
    elif mode == 1:      # heavy tail with exact zeros
        x = rng.standard_t(2.0, size=(T, I)).astype(np.float32) * np.float32(10.0 ** rng.uniform(-3, 1.5))
        x[rng.random((T, I)) < 0.1] = 0
    elif mode == 2:      # an outlier channel and an outlier token
        x = rng.standard_normal((T, I)).astype(np.float32)
        x[:, rng.integers(I)] *= 100
        x[rng.integers(T), :] *= 50
    else:                # powers of two only
        x = np.ldexp(np.float32(1.0), rng.integers(-10, 8, size=(T, I))).astype(np.float32)
        x *= rng.choice([-1.0, 1.0], size=(T, I)).astype(np.float32)
    if rng.random() < 0.2:
        x[rng.integers(T), :] = 0
    if rng.random() < 0.2:
        x[:, rng.integers(I)] = 0
    x = np.clip(x, -60000.0, 60000.0)                      # finite in fp16 too
    theta = float(rng.choice([1.0, 1.0, 0.5, 2.0, 3.7]))
    return dtype, bits, alpha, theta, wl.to_bits(x, dtype)


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_cases_through_every_quantizer(cq, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    for case in range(40):
        dtype, bits, alpha, theta, X = draw_case(rng)
        T, I = X.shape
        where = (seed, case, dtype, T, I, bits, alpha, theta)
        Xd = to_dev(X, dtype)
        r = cq.quantize_act(Xd, alpha, bits)
        parity.check_act(X, dtype, alpha, bits, t=r.t.cpu().numpy(), c=r.c.cpu().numpy(), a=r.row_scale.cpu().numpy(),
                         b=r.col_scale.cpu().numpy(), codes=r.codes.cpu().numpy(), deq=bits_of(r.deq),
                         zero_count=int(r.zero_count.item()))
        want, removed, k_pt, k_cq = orc.remove_kernel(X, dtype, alpha, bits, theta)
        out, counts = cq.remove_kernel(Xd, alpha, bits, theta)
        assert counts.cpu().tolist() == [removed, k_pt, k_cq], where
        assert np.array_equal(bits_of(out), want), where
        t, c = cq.absmax_rows_cols(Xd)
        assert int(cq.kernel_count_x(Xd, alpha, bits, t, c).item()) == k_cq, where
        ref = orc.quantize_weight_per_channel(X, dtype, bits)
        w = cq.quantize_weight_per_channel(Xd, bits)
        parity.check_weight(X, dtype, bits, scale=w.scale.cpu().numpy(), codes=w.codes.cpu().numpy(), deq=bits_of(w.deq),
                            zero_count=int(w.zero_count.item()), ref=ref)
        if I % 128 == 0:
            refg = orc.quantize_weight_groupwise(X, dtype, bits, 128)
            g = cq.quantize_weight_groupwise(Xd, 128, bits)
            parity.check_weight(X, dtype, bits, scale=g.scale.cpu().numpy(), codes=g.codes.cpu().numpy(),
                                deq=bits_of(g.deq), zero_count=int(g.zero_count.item()), ref=refg)
    assert cq.stage_fault() == 0
