"""The guard-band helper itself, on CPU tensors: an untouched arena passes, a store one byte past a payload (or
before it) is reported with the neighbouring buffer's name."""
from __future__ import annotations

import pytest
import torch

import guards


def _arena():
    ar = guards.Arena("cpu")
    ar.add("a", (3, 5), torch.float32)
    ar.add("b", 7, torch.int8, skew=3)
    ar.add("z", (), torch.int64)
    ar.add("empty", (0, 64), torch.int16)
    return ar.build()


def test_untouched_arena_passes_and_payloads_are_writable():
    ar = _arena()
    ar["a"].fill_(1.0)
    ar["b"].fill_(-1)
    ar["z"].fill_(7)
    ar.check("clean")
    assert ar["a"].shape == (3, 5) and ar["empty"].numel() == 0 and ar["z"].dim() == 0


@pytest.mark.parametrize("name,delta", [("a", 0), ("b", 0), ("z", 0), ("a", -1), ("b", -1)])
def test_a_store_just_outside_a_payload_is_reported(name, delta):
    ar = _arena()
    span = {n: (s, e) for n, s, e in ar._spans}[name]
    where = span[1] if delta == 0 else span[0] - 1        # first byte after / last byte before the payload
    ar.buf[where] = 0
    with pytest.raises(AssertionError) as e:
        ar.check("planted")
    assert name in str(e.value)
