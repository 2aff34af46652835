"""The weight kernels form fl32(x / s) under one scale per row or group without a division per element (one exact
reciprocal per row, two fused multiply-adds per element).  That this equals the IEEE quotient for every element and
every scale they can meet is checked here exhaustively, in plain C on the host (tests/native/exact_quotient_check.c)."""
from __future__ import annotations

import os
import subprocess
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))


def test_residual_corrected_division_is_the_ieee_quotient_for_every_16_bit_pair():
    src = os.path.join(HERE, "native", "exact_quotient_check.c")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "exact_quotient_check")
        subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-o", exe, src, "-lm"], check=True)
        out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout
    assert "pairs 8380418 mismatches 0" in out.stdout
