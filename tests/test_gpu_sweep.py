"""Layers of the 80-layer LLaMA-70B-shaped sweep at full size: every output of the 8 activation calls and the 6 weight
calls of a layer is compared with the oracle element by element (the whole sweep: tests/sweep_parity.py)."""
from __future__ import annotations

import pytest
import torch

pytestmark = pytest.mark.gpu

from sweep_parity import check_layer  # noqa: E402  (tests/ is on sys.path under pytest's rootdir conftest)


@pytest.mark.parametrize("layer", list(range(4, 80, 8)))
def test_sweep_layer_matches_the_oracle(cq, layer):
    rec = check_layer(layer, time_calls=False)
    assert rec["elements_compared"] == 2 * (3 * 2048 * 8192 + 2048 * 28672 + 2 * 8192 * 28672 + 8192 * 8192)
    assert rec["differences"] == 0
    assert cq.stage_fault() == 0
