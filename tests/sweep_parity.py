"""The 80-layer LLaMA-70B-shaped sweep with every output compared against the CPU oracle.

    python tests/sweep_parity.py --layers 80 [--stride 1] [--iters 5] [--table profiles/<name>.md]

Per layer: the four linear-layer input activations (2048 x 8192 three times, 2048 x 28672; bf16, Laplace values
with 8 outlier channels x50) are cross-quantized to INT8 and INT4 (alpha = 0.15) and the three weights
(8192 x 8192, 8192 x 28672, 28672 x 8192; bf16 N(0, 0.02^2)) are quantized per output channel to INT8 and INT4
through the public calls.  Every output of every call (absmax vectors, scale vectors, codes, 16-bit dequantized
matrix, zero-code count) is compared element by element with the oracle, which sees the same bytes; inputs are
generated per layer and dropped, so host memory holds one matrix at a time (plus the next one being drawn).
One JSON object per layer: quantizer time (sum of the 14 calls' mean CUDA-event times, L2 flushed by a 256 MiB read before each),
the kernel proportions (Definition 1; Section 4.2 averages them over all linear-layer inputs), the number of
differing elements (must be 0) and the oracle's wall time on the host cores.  This file lives under tests/
because it runs the oracle; the product package never does.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

ALPHA = 0.15


def _differences(got: np.ndarray, want: np.ndarray) -> int:
    """Number of positions whose bit patterns differ (shapes must agree)."""
    got, want = np.ascontiguousarray(got), np.ascontiguousarray(want)
    assert got.shape == want.shape and got.dtype.itemsize == want.dtype.itemsize, (got.shape, want.shape)
    width = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[got.dtype.itemsize]
    return int(np.count_nonzero(got.view(width) != want.view(width)))


def _inputs(layer: int):
    """The seven inputs of one layer, in the order they are processed: ('act', k, config) x 4, ('weight', k, shape) x 3."""
    from paper_2410_07505_b200 import workloads as wl
    for k in range(4):
        yield ("act", k, wl.sweep_activation_config(layer, k))
    for k in range(3):
        yield ("weight", k, wl.SWEEP_WEIGHT_SHAPES[k])


def _generate(layer: int, kind: str, k: int, what):
    from paper_2410_07505_b200 import workloads as wl
    return wl.generate_activation(what) if kind == "act" else wl.sweep_weight(layer, k, shape=what)


def check_layer(layer: int, *, iters: int = 5, time_calls: bool = True, flush=None, pool: ThreadPoolExecutor | None = None,
                weight_shapes=None, tokens: int | None = None) -> dict:
    """Run one layer of the sweep through the CUDA library, compare everything with the oracle, time the calls.

    `weight_shapes` / `tokens` shrink the layer (for quick checks); the defaults are the full configuration.
    Returns the per-layer record; `differences` is the total number of differing output elements.
    """
    import torch

    from oracle import cq_oracle as orc
    from oracle import parity
    from paper_2410_07505_b200 import cq, sweep, workloads as wl

    own_pool = pool is None
    evict = flush.read if flush is not None else None
    pool = pool or ThreadPoolExecutor(max_workers=1)
    todo = list(_inputs(layer))
    if tokens is not None:
        todo = [(kind, k, (wl.sweep_activation_config(layer, k, tokens) if kind == "act" else what)) for kind, k, what in todo]
    if weight_shapes is not None:
        todo = [(kind, k, (weight_shapes[k] if kind == "weight" else what)) for kind, k, what in todo]
    rec = {"layer": layer, "act_us": [], "weight_us": [], "kernel_proportion_int8_each": [],
           "kernel_proportion_int4_each": [], "weight_kernel_proportion_int8_each": [],
           "weight_kernel_proportion_int4_each": [], "differences": 0, "elements_compared": 0, "oracle_s": 0.0}
    pending = pool.submit(_generate, layer, *todo[0])
    for n, (kind, k, what) in enumerate(todo):
        M = pending.result()
        if n + 1 < len(todo):
            pending = pool.submit(_generate, layer, *todo[n + 1])
        Md = sweep._dev(M, "bf16")
        R, C = M.shape
        for bits in (8, 4):
            if kind == "act":
                buf = cq.ActBuffers(R, C, Md.dtype, bits)
                r = cq.quantize_act(Md, ALPHA, bits, buffers=buf)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                ref = orc.quantize_act(M, "bf16", ALPHA, bits, want_deq32=False, want_deq16=True)
                rec["oracle_s"] += time.perf_counter() - t0
                got_codes = r.codes.cpu().numpy()
                got_codes = parity.unpack_int4(got_codes, R, C) if bits == 4 else got_codes
                zc = int(r.zero_count.item())
                diffs = (_differences(r.t.cpu().numpy(), ref.t) + _differences(r.c.cpu().numpy(), ref.c) +
                         _differences(r.row_scale.cpu().numpy(), ref.a) + _differences(r.col_scale.cpu().numpy(), ref.b) +
                         _differences(got_codes, ref.codes) +
                         _differences(r.deq.view(torch.int16).cpu().numpy().view(np.uint16), ref.deq16) +
                         int(zc != ref.zero_count))
                rec["kernel_proportion_int%d_each" % bits].append(zc / (R * C))
                if time_calls:
                    rec["act_us"].append(round(sweep._time(lambda: cq.quantize_act(Md, ALPHA, bits, buffers=buf), evict, iters), 1))
                del buf, r
            else:
                out = cq.quantize_weight_per_channel(Md, bits)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                ref = orc.quantize_weight_per_channel(M, "bf16", bits, want_deq32=False, want_deq16=True)
                rec["oracle_s"] += time.perf_counter() - t0
                got_codes = out.codes.cpu().numpy()
                got_codes = parity.unpack_int4(got_codes, R, C) if bits == 4 else got_codes
                zc = int(out.zero_count.item())
                diffs = (_differences(out.scale.cpu().numpy(), ref.scale) + _differences(got_codes, ref.codes) +
                         _differences(out.deq.view(torch.int16).cpu().numpy().view(np.uint16), ref.deq16) +
                         int(zc != ref.zero_count))
                rec["weight_kernel_proportion_int%d_each" % bits].append(zc / (R * C))
                if time_calls:
                    rec["weight_us"].append(round(sweep._time(lambda: cq.quantize_weight_per_channel(Md, bits, out=out), evict, iters), 1))
                del out
            rec["differences"] += diffs
            rec["elements_compared"] += R * C
            del ref, got_codes
        del Md, M
    if own_pool:
        pool.shutdown()
    p8 = rec["kernel_proportion_int8_each"]
    p4 = rec["kernel_proportion_int4_each"]
    rec["kernel_proportion_int8_mean"] = sum(p8) / len(p8)
    rec["kernel_proportion_int4_mean"] = sum(p4) / len(p4)
    rec["quantizer_us"] = round(sum(rec["act_us"]) + sum(rec["weight_us"]), 1)
    rec["oracle_s"] = round(rec["oracle_s"], 2)
    return rec


def write_table(path: str, records: list, summary: dict, command: str) -> None:
    """The per-layer table as markdown (a summary for profiles/, a few KB)."""
    lines = [
        "# 80-layer LLaMA-70B-shaped sweep at 2048 tokens: quantizer time, kernel proportion and parity per layer",
        "",
        "Command (one B200; prints one JSON object per layer, this table is its output reformatted):",
        "",
        f"    {command}",
        "",
        "Per layer: 4 activations (2048x8192 x3, 2048x28672; bf16 Laplace, 8 outlier channels x50, alpha = 0.15) x {INT8, INT4}",
        "through `cq_quantize_act` (t, c, scale vectors, codes, bf16 dequantized, count) and 3 weights (8192x8192, 8192x28672,",
        "28672x8192; bf16 N(0, 0.02^2)) x {INT8, INT4} through `cq_quantize_weight_per_channel` (scale, codes, bf16 dequantized,",
        "count).  Time = sum of the 14 calls' mean CUDA-event times, L2 flushed (a 256 MiB buffer read twice) before every call.  Every output element of every",
        "call is compared with the CPU oracle on the same bytes; `diff` is the number of differing elements.",
        "",
        f"* layers run: {summary['layers_run']}, elements compared: {summary['elements_compared']:,}, differing: "
        f"**{summary['differences']}**",
        f"* quantizer time, all layers: **{summary['end_to_end_quantizer_ms']:.2f} ms** on the GPU "
        f"(mean {summary['mean_layer_us']:.1f} us per layer, min {summary['min_layer_us']:.1f}, max {summary['max_layer_us']:.1f}); "
        f"the oracle took {summary['oracle_s']:.1f} s of wall time for the same work on {summary['oracle_threads']} host threads",
        f"* kernel proportion averaged over all linear-layer inputs (Section 4.2): INT8 {summary['kernel_proportion_int8_mean']:.4%}, "
        f"INT4 {summary['kernel_proportion_int4_mean']:.4%}",
        f"* SM clock during the run: median {summary['clocks'].get('sm_mhz')} MHz of {summary['clocks'].get('sm_max_mhz')}, "
        f"throttle reasons {summary['clocks'].get('reasons')}",
        "",
        "| layer | quantizer us | activations us (INT8, INT4 per input) | weights us (INT8, INT4 per shape) | INT8 kernel proportion of the 4 inputs | mean INT8 | mean INT4 | diff |",
        "|---|---|---|---|---|---|---|---|",
    ]
    for r in records:
        lines.append("| {layer} | {q:.1f} | {a} | {w} | {p} | {m8:.3%} | {m4:.3%} | {d} |".format(
            layer=r["layer"], q=r["quantizer_us"], a=" ".join(f"{x:.1f}" for x in r["act_us"]),
            w=" ".join(f"{x:.1f}" for x in r["weight_us"]),
            p=" ".join(f"{x:.3%}" for x in r["kernel_proportion_int8_each"]),
            m8=r["kernel_proportion_int8_mean"], m4=r["kernel_proportion_int4_mean"], d=r["differences"]))
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=80)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--table", default="", help="also write the per-layer table as markdown to this path")
    args = ap.parse_args()

    import torch

    from oracle import build as oracle_build, cq_oracle as orc
    from paper_2410_07505_b200 import build as cuda_build, clocks, cq

    oracle_build.build()
    cuda_build.build()
    cq.lib()
    from paper_2410_07505_b200 import sweep
    flush = sweep.L2Flush()
    records = []
    with ThreadPoolExecutor(max_workers=1) as pool, clocks.for_current_device(0.05) as clk:
        for layer in range(0, args.layers, max(1, args.stride)):
            rec = check_layer(layer, iters=args.iters, flush=flush, pool=pool)
            records.append(rec)
            print(json.dumps(rec), flush=True)
    n = len(records)
    us = [r["quantizer_us"] for r in records]
    summary = {
        "layers_run": n, "end_to_end_quantizer_ms": sum(us) / 1e3, "mean_layer_us": sum(us) / n,
        "min_layer_us": min(us), "max_layer_us": max(us),
        "differences": sum(r["differences"] for r in records),
        "elements_compared": sum(r["elements_compared"] for r in records),
        "kernel_proportion_int8_mean": sum(r["kernel_proportion_int8_mean"] for r in records) / n,
        "kernel_proportion_int4_mean": sum(r["kernel_proportion_int4_mean"] for r in records) / n,
        "oracle_s": sum(r["oracle_s"] for r in records), "oracle_threads": orc.num_threads(),
        "stage_fault": cq.stage_fault(), "clocks": clk.summary(),
    }
    print(json.dumps(summary), flush=True)
    if args.table:
        cmd = "python tests/sweep_parity.py --layers %d%s --iters %d --table %s" % (
            args.layers, f" --stride {args.stride}" if args.stride != 1 else "", args.iters, args.table)
        write_table(args.table, records, summary, cmd)
    return 0 if summary["differences"] == 0 and summary["stage_fault"] == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
