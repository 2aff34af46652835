"""Per-configuration timing table and the 80-layer LLaMA-70B-shaped sweep.

    python -m paper_2410_07505_b200.sweep                 # every activation config x bit width, 3 weight shapes
    python -m paper_2410_07505_b200.sweep --layers 80     # plus the per-layer sweep (inputs generated per layer)

Times are CUDA-event means of the public calls with the L2 flushed before every call by reading a 256 MiB buffer
twice (clean lines: the cold number), by a 256 MiB write (126 MB of dirty lines whose write-back competes with
the call's first pass) and back to back without a flush.  GB/s uses the algorithmic byte counts:
activations 2+2+codes+2 bytes per element (X read twice; the single-read figure drops one read, for
matrices L2 can hold), weights 2+codes+2 (row read once).  Every row carries the SM clock sampled while
it was timed.  One JSON object per line.
"""
from __future__ import annotations

import argparse
import json
import statistics

import numpy as np
import torch

from . import clocks
from . import cq
from . import workloads as wl

TORCH_DT = {"f16": torch.float16, "bf16": torch.bfloat16}


def _dev(bits: np.ndarray, dtype: str) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(TORCH_DT[dtype]).cuda()


class L2Flush:
    """Untimed eviction of L2 between timed calls: `read` leaves clean lines behind, `write` dirty ones."""

    def __init__(self, nbytes: int = 256 << 20, device="cuda"):
        self.buf = torch.zeros(nbytes, dtype=torch.uint8, device=device)
        self.words = self.buf.view(torch.int64)      # summed as it is (a narrower type would be widened into a temporary first)
        self.sum = torch.zeros((), dtype=torch.int64, device=device)

    def read(self) -> None:
        for _ in range(2):        # a single pass over 256 MiB still leaves some of the previous call's dirty lines in L2
            torch.sum(self.words, dim=0, out=self.sum)

    def write(self) -> None:
        self.buf.zero_()


def _time(fn, flush, iters: int) -> float:
    """Mean CUDA-event time of `fn` in microseconds; `flush` (a callable or None) runs untimed before every call.
    (The event clock ticks in steps of about two microseconds here, so a mean resolves what a median cannot.)"""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    for a, b in ev:
        if flush is not None:
            flush()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return statistics.fmean(a.elapsed_time(b) for a, b in ev) * 1e3     # microseconds


def time_activation(Xd: torch.Tensor, bits: int, alpha: float, flush, iters: int) -> dict:
    T, I = Xd.shape
    buf = cq.ActBuffers(T, I, Xd.dtype, bits)
    with clocks.for_current_device() as clk:
        us_cold = _time(lambda: cq.quantize_act(Xd, alpha, bits, buffers=buf), flush.read, iters)
        us_dirty = _time(lambda: cq.quantize_act(Xd, alpha, bits, buffers=buf), flush.write, iters)
        us_warm = _time(lambda: cq.quantize_act(Xd, alpha, bits, buffers=buf), None, iters)
    n = T * I
    per_elem = 2 + 2 + (1 if bits == 8 else 0.5) + 2
    return {"us_l2_flushed": round(us_cold, 1), "us_write_flushed": round(us_dirty, 1), "us_back_to_back": round(us_warm, 1),
            "sm_mhz": clk.summary()["sm_mhz"],
            "gbs_l2_flushed": round(per_elem * n / us_cold / 1e3, 1),
            "gbs_single_read_accounting": round((per_elem - 2) * n / us_cold / 1e3, 1),
            "elements_per_s": round(n / us_cold * 1e6), "kernel_proportion": int(buf.zero_count.item()) / n}


def time_weight(Wd: torch.Tensor, bits: int, flush, iters: int) -> dict:
    out = cq.quantize_weight_per_channel(Wd, bits)
    with clocks.for_current_device() as clk:
        us = _time(lambda: cq.quantize_weight_per_channel(Wd, bits, out=out), flush.read, iters)
    n = Wd.numel()
    per_elem = 2 + (1 if bits == 8 else 0.5) + 2
    return {"us_l2_flushed": round(us, 1), "sm_mhz": clk.summary()["sm_mhz"], "gbs": round(per_elem * n / us / 1e3, 1),
            "kernel_proportion": int(out.zero_count.item()) / n}


def time_extra_ops(Xd: torch.Tensor, alpha: float, flush, iters: int) -> dict:
    """Remove-Kernel operator, Table 1 indicators and the count-only pass on one activation matrix."""
    T, I = Xd.shape
    n = T * I
    ws = torch.empty(cq.workspace_bytes(T, I), dtype=torch.uint8, device=Xd.device)
    r = cq.quantize_act(Xd, alpha, 8)
    t, c = cq.absmax_rows_cols(Xd)
    us_rm = _time(lambda: cq.remove_kernel(Xd, alpha, 8, 1.0, ws), flush.read, iters)
    us_ind = _time(lambda: cq.case_indicators(r), flush.read, iters)
    us_cnt = _time(lambda: cq.kernel_count_x(Xd, alpha, 8, t, c, ws), flush.read, iters)
    us_abs = _time(lambda: cq.absmax_rows_cols(Xd), flush.read, iters)
    us_abs_ws = _time(lambda: cq.absmax_rows_cols(Xd, workspace=ws, out=(t, c)), flush.read, iters)
    deq = torch.empty((T, I), dtype=Xd.dtype, device=Xd.device)
    cnt = torch.zeros((), dtype=torch.int64, device=Xd.device)
    us_deq = _time(lambda: cq.dequantize(r.codes, 8, T, I, r.row_scale, r.col_scale, Xd.dtype, out=deq), flush.read, iters)
    us_kc = _time(lambda: cq.kernel_count(r.codes, 8, T, I, count=cnt), flush.read, iters)
    _, counts = cq.remove_kernel(Xd, alpha, 8, 1.0, ws)
    ind = cq.case_indicators(r).cpu().tolist()
    cnt = counts.cpu().tolist()
    return {"remove_kernel_us": round(us_rm, 1), "remove_kernel_gbs": round(6 * n / us_rm / 1e3, 1),
            "case_indicators_us": round(us_ind, 1), "kernel_count_x_us": round(us_cnt, 1),
            "absmax_rows_cols_us": round(us_abs, 1), "absmax_gbs": round(2 * n / us_abs / 1e3, 1),
            "absmax_with_workspace_us": round(us_abs_ws, 1),
            "dequantize_us": round(us_deq, 1), "dequantize_gbs": round(3 * n / us_deq / 1e3, 1),
            "kernel_count_us": round(us_kc, 1), "kernel_count_gbs": round(n / us_kc / 1e3, 1),
            "kernel_proportion_per_token": cnt[1] / n, "kernel_proportion_crossquant": cnt[2] / n,
            "share_c_ge_t": ind[0] / n, "share_bound_smaller": ind[1] / n}


def time_whole_layer(layer: int, alpha: float, iters: int) -> dict:
    """One layer of the 80-layer sweep the way a pipeline would run it: the seven inputs resident on the device, the 14
    quantizer calls (4 activations and 3 weights, INT8 and INT4 each) issued back to back on one stream between ONE pair
    of events -- no flush, no per-call event latency -- and the same 14 calls replayed from one CUDA graph."""
    acts = [_dev(wl.generate_activation(wl.sweep_activation_config(layer, k)), "bf16") for k in range(4)]
    weights = [_dev(wl.sweep_weight(layer, k), "bf16") for k in range(3)]
    abuf = {(k, bits): cq.ActBuffers(X.shape[0], X.shape[1], X.dtype, bits) for k, X in enumerate(acts) for bits in (8, 4)}
    wout = {(k, bits): cq.quantize_weight_per_channel(W, bits) for k, W in enumerate(weights) for bits in (8, 4)}

    def layer_calls():
        for k, X in enumerate(acts):
            for bits in (8, 4):
                cq.quantize_act(X, alpha, bits, buffers=abuf[(k, bits)])
        for k, W in enumerate(weights):
            for bits in (8, 4):
                cq.quantize_weight_per_channel(W, bits, out=wout[(k, bits)])

    with clocks.for_current_device() as clk:
        us_calls = _time(layer_calls, None, iters)
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            layer_calls()
        us_graph = _time(graph.replay, None, iters)
    elements = sum(X.numel() for X in acts) + sum(W.numel() for W in weights)
    return {"layer": layer, "whole_layer_back_to_back_us": round(us_calls, 1), "whole_layer_graph_replay_us": round(us_graph, 1),
            "calls": 14, "elements_per_bit_width": elements, "sm_mhz": clk.summary()["sm_mhz"]}


def time_decode_shapes(flush, iters: int) -> None:
    """Decode-sized matrices: CUDA-event time of one call after an L2 flush, wall time per call of 200 calls issued
    back to back (host included), for the single-launch path and the three launches, and per replay of a graph."""
    import time
    for T, I in ((1, 4096), (16, 4096), (16, 8192), (32, 2048), (128, 768), (64, 2048), (32, 4096), (64, 8192)):
        Xd = _dev(wl.small_matrix(T, I, "bf16", 3, outlier_cols=4), "bf16")
        buf = cq.ActBuffers(T, I, Xd.dtype, 8)
        row = {"shape": [T, I], "dtype": "bf16", "bits": 8}
        for key, no_small in (("one_launch", 0), ("three_launches", 1)):
            cq.set_tuning("no_small", no_small)
            cold = _time(lambda: cq.quantize_act(Xd, 0.15, 8, buffers=buf), flush.read, iters)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(200):
                cq.quantize_act(Xd, 0.15, 8, buffers=buf)
            torch.cuda.synchronize()
            row[key] = {"us_l2_flushed": round(cold, 1), "us_per_call_back_to_back": round((time.perf_counter() - t0) / 200 * 1e6, 1)}
        cq.set_tuning("no_small", 0)
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            cq.quantize_act(Xd, 0.15, 8, buffers=buf)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(200):
            graph.replay()
        torch.cuda.synchronize()
        row["graph_replay_us"] = round((time.perf_counter() - t0) / 200 * 1e6, 1)
        print(json.dumps(row), flush=True)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--layers", type=int, default=0, help="layers of the 80-layer sweep to run (0 = skip)")
    ap.add_argument("--alpha", type=float, default=0.15)
    ap.add_argument("--whole-layer", action="store_true", help="with --layers: also time each layer's 14 calls issued back to back "
                    "between ONE pair of events (all seven inputs resident, no flush), and replayed from a CUDA graph")
    ap.add_argument("--decode", action="store_true", help="time decode-sized matrices through the single-launch path, "
                    "the three launches and a CUDA-graph replay, then exit")
    ap.add_argument("--tune", action="append", default=[], metavar="KEY=VALUE",
                    help="launch-shape knob to set before timing (see cq_set_tuning), e.g. no_pdl=1; may be repeated")
    ap.add_argument("--only", default="", help="comma-separated config names (e.g. llama70b_mlp,weight_8192x28672): "
                    "time only these (keeps a profiler capture short)")
    args = ap.parse_args()
    only = set(filter(None, args.only.split(",")))
    cq.lib()
    for kv in args.tune:
        key, _, value = kv.partition("=")
        cq.set_tuning(key, int(value))
    flush = L2Flush()
    if args.decode:
        time_decode_shapes(flush, args.iters)
        return

    for name, cfg in wl.ACT_CONFIGS.items():
        if only and name not in only:
            continue
        Xd = _dev(wl.generate_activation(cfg), cfg.dtype)
        for bits in cfg.bits:
            for alpha in cfg.alphas:
                row = {"config": name, "shape": [cfg.T, cfg.I], "dtype": cfg.dtype, "bits": bits, "alpha": alpha}
                row.update(time_activation(Xd, bits, alpha, flush, args.iters))
                print(json.dumps(row), flush=True)
        if name != "tiny":
            row = {"config": name, "shape": [cfg.T, cfg.I], "dtype": cfg.dtype, "ops": "diagnostics", "alpha": args.alpha}
            row.update(time_extra_ops(Xd, args.alpha, flush, args.iters))
            print(json.dumps(row), flush=True)
        del Xd
    for k, shape in enumerate(wl.SWEEP_WEIGHT_SHAPES):
        if only and f"weight_{shape[0]}x{shape[1]}" not in only:
            continue
        Wd = _dev(wl.sweep_weight(0, k), "bf16")
        for bits in (8, 4):
            row = {"config": f"weight_{shape[0]}x{shape[1]}", "shape": list(shape), "dtype": "bf16", "bits": bits}
            row.update(time_weight(Wd, bits, flush, args.iters))
            print(json.dumps(row), flush=True)
        out = cq.quantize_weight_groupwise(Wd, 128, 4)
        with clocks.for_current_device() as clk:
            us = _time(lambda: cq.quantize_weight_groupwise(Wd, 128, 4, out=out), flush.read, args.iters)
        print(json.dumps({"config": f"weight_{shape[0]}x{shape[1]}_g128", "shape": list(shape), "dtype": "bf16", "bits": 4,
                          "us_l2_flushed": round(us, 1), "sm_mhz": clk.summary()["sm_mhz"], "gbs": round(4.5 * Wd.numel() / us / 1e3, 1),
                          "kernel_proportion": int(out.zero_count.item()) / Wd.numel()}), flush=True)
        del Wd, out

    total_us = 0.0
    for layer in range(args.layers):
        if args.whole_layer:
            print(json.dumps(time_whole_layer(layer, args.alpha, max(5, args.iters // 3))), flush=True)
        props = []
        layer_us = 0.0
        for k in range(4):
            cfg = wl.sweep_activation_config(layer, k)
            Xd = _dev(wl.generate_activation(cfg), cfg.dtype)
            for bits in (8, 4):
                r = time_activation(Xd, bits, args.alpha, flush, max(5, args.iters // 3))
                layer_us += r["us_l2_flushed"]
                if bits == 8:
                    props.append(r["kernel_proportion"])
            del Xd
        for k in range(3):
            Wd = _dev(wl.sweep_weight(layer, k), "bf16")
            for bits in (8, 4):
                layer_us += time_weight(Wd, bits, flush, max(5, args.iters // 3))["us_l2_flushed"]
            del Wd
        total_us += layer_us
        print(json.dumps({"layer": layer, "quantizer_us": round(layer_us, 1),
                          "kernel_proportion_int8_mean": sum(props) / len(props),
                          "kernel_proportion_int8_each": props}), flush=True)
    if args.layers:
        print(json.dumps({"layers": args.layers, "end_to_end_quantizer_ms": round(total_us / 1e3, 3)}))


if __name__ == "__main__":
    main()
