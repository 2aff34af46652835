"""The five benchmark configurations at full size, in the launch configuration the benchmark
times, against the oracle on every element (the C oracle finishes each matrix in seconds)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import cq_oracle as orc
from oracle import parity
from paper_2410_07505_b200 import workloads as wl

from test_gpu_parity import bits_of, to_dev

pytestmark = pytest.mark.gpu


def _check_config(cq, X, cfg):
    Xd = to_dev(X, cfg.dtype)
    T, I = X.shape
    for bits in cfg.bits:
        buf = cq.ActBuffers(T, I, Xd.dtype, bits)
        for alpha in cfg.alphas:
            r = cq.quantize_act(Xd, alpha, bits, buffers=buf)
            torch.cuda.synchronize()
            rep = parity.check_act(X, cfg.dtype, alpha, bits, t=r.t.cpu().numpy(), c=r.c.cpu().numpy(),
                                   a=r.row_scale.cpu().numpy(), b=r.col_scale.cpu().numpy(),
                                   codes=r.codes.cpu().numpy(), deq=bits_of(r.deq),
                                   zero_count=int(r.zero_count.item()))
            assert rep.code_mismatches <= 1e-6 * T * I
            assert abs(r.kernel_proportion() - rep.kernel_proportion) <= 1e-6
        del buf


@pytest.mark.parametrize("name", list(wl.ACT_CONFIGS))
def test_activation_config(cq, name):
    X, cfg = wl.activation(name)
    _check_config(cq, X, cfg)


def test_headline_config_fp32_dequant_and_count_only(cq):
    X, cfg = wl.activation(wl.HEADLINE)
    Xd = to_dev(X, cfg.dtype)
    ref = orc.quantize_act(X, cfg.dtype, 0.15, 8, want_deq16=False)
    r = cq.quantize_act(Xd, 0.15, 8, codes=False, deq_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(r.zero_count.item()) == ref.zero_count
    # sampled rows of the fp32 output (the full 470 MB comparison adds nothing over the bf16 one)
    rows = np.linspace(0, X.shape[0] - 1, 64).astype(np.int64)
    got = r.deq[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert np.array_equal(got.view(np.uint32), ref.deq32[rows].view(np.uint32))
    t, c = cq.absmax_rows_cols(Xd)
    assert int(cq.kernel_count_x(Xd, 0.15, 8, t, c).item()) == ref.zero_count


@pytest.mark.parametrize("layer", [0, 79])
def test_sweep_layer_activations(cq, layer):
    for k in range(4):
        cfg = wl.sweep_activation_config(layer, k)
        X = wl.generate_activation(cfg)
        _check_config(cq, X, cfg)


@pytest.mark.parametrize("k", [0, 1, 2])
def test_sweep_layer_weights(cq, k):
    W = wl.sweep_weight(0, k)
    Wd = to_dev(W, "bf16")
    for bits in (8, 4):
        ref = orc.quantize_weight_per_channel(W, "bf16", bits, want_deq32=False)
        r = cq.quantize_weight_per_channel(Wd, bits)
        torch.cuda.synchronize()
        parity.check_weight(W, "bf16", bits, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(),
                            deq=bits_of(r.deq), zero_count=int(r.zero_count.item()), ref=ref)
        del r


def test_sweep_weight_groupwise_g128(cq):
    """W4-g128 on a full-size sweep weight (the paper's W4A8-g128 setting)."""
    W = wl.sweep_weight(0, 1)
    Wd = to_dev(W, "bf16")
    ref = orc.quantize_weight_groupwise(W, "bf16", 4, 128)
    r = cq.quantize_weight_groupwise(Wd, 128, 4)
    torch.cuda.synchronize()
    parity.check_weight(W, "bf16", 4, scale=r.scale.cpu().numpy(), codes=r.codes.cpu().numpy(),
                        deq=bits_of(r.deq), zero_count=int(r.zero_count.item()), ref=ref)


def test_diagnostics_operators_at_full_size(cq):
    """Remove Kernel (with both kernel counts) and the Table 1 indicators on a full-size config."""
    X, cfg = wl.activation("llama70b_attn")
    Xd = to_dev(X, cfg.dtype)
    want, removed, k_pt, k_cq = orc.remove_kernel(X, cfg.dtype, 0.15, 8, 1.0)
    out, counts = cq.remove_kernel(Xd, 0.15, 8, 1.0)
    torch.cuda.synchronize()
    assert counts.cpu().tolist() == [removed, k_pt, k_cq]
    assert np.array_equal(bits_of(out), want)
    r = cq.quantize_act(Xd, 0.15, 8)
    ref = orc.quantize_act(X, cfg.dtype, 0.15, 8, want_deq32=False, want_deq16=False)
    assert tuple(cq.case_indicators(r).cpu().tolist()) == orc.case_indicators(ref.t, ref.c, ref.a, ref.b, 8)
    assert int(r.zero_count.item()) == k_cq


def test_crossquant_on_a_weight_matrix(cq):
    """CrossQuant applied to weights (Appendix B: alpha_W = 0.55 for OPT-66B W4A4) is the activation entry point on W."""
    W = wl.sweep_weight(0, 0)
    Wd = to_dev(W, "bf16")
    r = cq.quantize_act(Wd, 0.55, 4)
    torch.cuda.synchronize()
    parity.check_act(W, "bf16", 0.55, 4, t=r.t.cpu().numpy(), c=r.c.cpu().numpy(), a=r.row_scale.cpu().numpy(),
                     b=r.col_scale.cpu().numpy(), codes=r.codes.cpu().numpy(), deq=bits_of(r.deq),
                     zero_count=int(r.zero_count.item()))


def test_no_bounded_wait_ever_gave_up(cq):
    """Collected after the full-size runs: the staged quantize pass never abandoned a wait on a row copy."""
    torch.cuda.synchronize()
    assert cq.stage_fault() == 0
