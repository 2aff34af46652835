#!/usr/bin/env python
"""Benchmark of the CrossQuant activation quantizer on B200.

One step = one full cq_quantize_act call (row/column absmax, scale vectors, INT8 codes, bf16
dequantized matrix, zero-code count) on the LLaMA-70B-MLP-shaped activation matrix
(4096 x 28672 bf16, Laplace values with 8 outlier channels x50, alpha = 0.15).  The metric is
algorithmic bytes per second: 7 bytes per element (two compulsory reads of X, one byte of
codes, two bytes of dequantized output) divided by the device time of the step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--mode replicas|row_sharded]

With N > 1 there is one rank per GPU: started by torchrun (RANK / LOCAL_RANK / WORLD_SIZE in the
environment) or, when the script is run directly, by the script itself, which re-launches itself under
torch.distributed.run on 127.0.0.1.  A world size that does not match --gpus, or fewer GPUs than ranks, is
an error, never a silent single-GPU run.  Default mode: every rank quantizes its own matrix of the same
shape -- the path has no exchange step, so the ranks are independent (weak scaling).  --mode row_sharded
measures the sharded variant instead: ONE matrix of the same shape with its tokens split over the ranks,
the column maxima combined by an all-reduce MAX between the passes (strong scaling).
`--impl reference` times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "CrossQuant act-quant GB/s and % of HBM roofline at LLaMA-70B-shaped X"
UNIT = "GB/s"
ALPHA = 0.15
BITS = 8
BYTES_PER_ELEMENT_STEP = 7.0        # X read twice (2+2) + int8 codes (1) + bf16 dequantized (2)
BYTES_PER_ELEMENT_QUANT_PASS = 5.0  # quantize pass alone: X (2) + codes (1) + dequantized (2)
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 256 << 20
E2E_STREAMS = 2              # a third stream changes nothing: the device-to-host copies already run back to back
HOOK_LAUNCHES = 64          # launches of the quantize pass timed inside real calls for the roofline object

# DRAM traffic of the quantize pass from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum
# per launch), valid only for the kernel sources whose digest is recorded with it.
NCU_TRAFFIC = {"sources_sha256": "f000b397e96a39f12525e40ed6ad30a3edcd77b8d232cc27ab255723a4cc0093",
               "bytes_per_launch": 528164352}   # 235,185,920 read + 292,978,432 written


def kernel_sources_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("cq_act.cu", "cq_common.cuh", "cq_passes.cuh"):
        with open(os.path.join(ROOT, "paper_2410_07505_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def rank_config(rank: int):
    from paper_2410_07505_b200 import workloads as wl
    cfg = wl.ACT_CONFIGS[wl.HEADLINE]
    if rank:
        cfg = dataclasses.replace(cfg, seed=cfg.seed + 100 * rank)
    return cfg


def max_over_ranks(local_ms: float, device: str) -> float:
    """Largest per-rank device time; every rank gets the same answer (one all-reduce MAX)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(elements_per_rank: int, steps: int, world: int, max_ms: float) -> float:
    """Aggregate algorithmic GB/s of `world` independent ranks over the slowest rank's time."""
    return BYTES_PER_ELEMENT_STEP * elements_per_rank * steps * world / (max_ms * 1e-3) / 1e9


def workload_name(cfg) -> str:
    return (f"{cfg.name} {cfg.T}x{cfg.I} bf16 (LLaMA-70B MLP input), INT{BITS} codes + bf16 dequant + zero count, "
            f"alpha={ALPHA}")


def run_reference(args) -> None:
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cq_oracle as orc
    from paper_2410_07505_b200 import workloads as wl
    cfg = rank_config(0)
    rows = 256
    sample_cfg = dataclasses.replace(cfg, T=rows)
    X = wl.generate_activation(sample_cfg)
    for _ in range(args.warmup):
        orc.quantize_act(X, cfg.dtype, ALPHA, BITS, want_deq32=False)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.quantize_act(X, cfg.dtype, ALPHA, BITS, want_deq32=False)
    dt = time.perf_counter() - t0
    value = BYTES_PER_ELEMENT_STEP * X.size * args.steps / dt / 1e9
    sample = f"first {rows} rows of the {cfg.T}x{cfg.I} matrix per step (oracle quantize_act: t, c, codes, bf16 dequant, count)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_row_sharded(args) -> None:
    """The sharded variant of the path (tokens of ONE matrix split over the ranks): per step every rank runs the
    absmax pass on its row block, the column maxima are combined by an all-reduce MAX (I floats, NCCL, into local
    memory), and every rank quantizes its block with its own t and the combined c; the kernel sizes are summed.
    Strong scaling: the matrix is the headline one whatever the number of ranks."""
    import torch
    import torch.distributed as dist

    from paper_2410_07505_b200 import build as cuda_build, clocks as clk, cq, sharded, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if local == 0:
        cuda_build.build()
    if world > 1:
        dist.barrier()
    cq.lib()
    cfg = rank_config(0)                                   # the same matrix on every rank: each keeps its rows
    X = wl.generate_activation(cfg)
    T, I = X.shape
    r0, r1 = sharded.shard_rows(T, world, rank)
    Xd = torch.from_numpy(np.ascontiguousarray(X[r0:r1]).view(np.int16)).view(torch.bfloat16).cuda()
    del X
    buf = cq.ActBuffers(r1 - r0, I, torch.bfloat16, BITS)
    flush_words = torch.zeros(L2_FLUSH_BYTES // 8, dtype=torch.int64, device="cuda")
    flush_sum = torch.zeros((), dtype=torch.int64, device="cuda")

    def step():
        return sharded.quantize_act_row_sharded(Xd, ALPHA, BITS, buffers=buf)

    def flush_l2():
        for _ in range(2):
            torch.sum(flush_words, dim=0, out=flush_sum)

    for _ in range(args.warmup):
        flush_l2()
        step()
    torch.cuda.synchronize()
    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    with clk.ClockSampler(local, str(torch.cuda.get_device_properties(local).uuid), period_s=0.002) as clocks:
        for a_, b_ in ev:
            flush_l2()
            a_.record()
            _, total = step()
            b_.record()
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = max_over_ranks(sum(a_.elapsed_time(b_) for a_, b_ in ev), "cuda")
    n = T * I
    value = BYTES_PER_ELEMENT_STEP * n * K / (total_ms * 1e-3) / 1e9          # the whole matrix per step, all ranks together
    if rank == 0:
        peak, peak_kind = measured_peak()
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "mode": "row_sharded",
            "config": {"workload": workload_name(cfg) + f", tokens split over {world} rank(s)",
                       "exchange": "all-reduce MAX of the column maxima (I floats) between the passes, all-reduce SUM of the "
                                   "kernel sizes; NCCL into local memory, no peer-memory operands",
                       "l2": "flushed between steps by reading a 256 MiB buffer twice, untimed",
                       "timing": "CUDA events per step on the launch stream, summed; max over ranks"},
            "fraction_of_hbm_roofline": value / (peak * world), "peak_kind": f"of {peak_kind}",
            "kernel_proportion": int(total.item()) / n, "clocks": clocks.summary(),
            "gpu_launches": 3 * K, "e2e": None}))
    if world > 1:
        dist.destroy_process_group()


def ensure_ranks(args, argv) -> None:
    """Make --gpus N mean N ranks.  Under a launcher (WORLD_SIZE set) the world size must equal N; run directly with
    N > 1, the script starts its own ranks: it replaces itself by torch.distributed.run (one node, rendezvous on
    127.0.0.1) running the same command line.  Never falls back to fewer ranks."""
    world = os.environ.get("WORLD_SIZE")
    if world is not None:
        if int(world) != args.gpus:
            sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}: refusing to run with another number of ranks")
        return
    if args.gpus == 1:
        return
    if args.gpus < 1:
        sys.exit("bench.py: --gpus must be at least 1")
    if not args.dry_run:
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            sys.exit(f"bench.py: --gpus {args.gpus} but only {have} CUDA device(s) are visible: refusing to run on fewer")
    os.environ.setdefault("NCCL_DEBUG", "INFO")         # the communicator log (transport, NVLS) goes to stderr with the run
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--local-addr", "127.0.0.1", os.path.abspath(__file__), *argv]
    sys.stdout.flush()
    os.execv(sys.executable, cmd)


def run_dry(args) -> None:
    """The rank plumbing alone, on the CPU (gloo): rendezvous, barrier, max over ranks, one JSON line from rank 0."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    seen = torch.zeros(world, dtype=torch.int64)
    seen[rank] = 1
    if world > 1:
        dist.all_reduce(seen)
    slowest = max_over_ranks(1.0 + rank, "cpu")
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ranks_seen": int(seen.sum()), "max_ms": slowest,
                          "mode": args.mode, "seeds": [rank_config(r).seed for r in range(world)]}))
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--mode", default="replicas", choices=["replicas", "row_sharded"],
                    help="replicas: one matrix per rank, no exchange (weak scaling, the headline); row_sharded: one matrix "
                         "with its tokens split over the ranks and an all-reduce MAX of the column maxima (strong scaling)")
    ap.add_argument("--dry-run", action="store_true", help="start the ranks, run the rank plumbing on the CPU (gloo) and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return
    ensure_ranks(args, sys.argv[1:])
    if args.dry_run:
        run_dry(args)
        return
    if args.mode == "row_sharded":
        run_row_sharded(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2410_07505_b200 import build as cuda_build, clocks as clk, cq, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if local == 0:
        cuda_build.build()
    if world > 1:
        dist.barrier()
    cq.lib()

    cfg = rank_config(rank)
    X = wl.generate_activation(cfg)
    T, I = X.shape
    n = T * I
    Xh = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16)
    Xd = Xh.cuda()
    buf = cq.ActBuffers(T, I, torch.bfloat16, BITS)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda").zero_()
    flush_words = flush.view(torch.int64)      # summed as it is: a narrower type would first be widened into a 512 MiB temporary
    flush_sum = torch.zeros((), dtype=torch.int64, device="cuda")

    def flush_l2(kind: str) -> None:
        """Untimed, between steps.  "read": a 256 MiB buffer read twice pushes X and the outputs out of L2 and leaves
        clean lines behind.  "write": a 256 MiB fill does the same but leaves 126 MB of dirty lines, whose write-back then
        competes with the step's first pass (reported beside the headline, not as it)."""
        if kind == "read":
            for _ in range(2):                        # one pass still leaves some of the last step's dirty output lines
                torch.sum(flush_words, dim=0, out=flush_sum)
        elif kind == "write":
            flush.zero_()

    def step():
        cq.quantize_act(Xd, ALPHA, BITS, buffers=buf)

    for _ in range(args.warmup):
        flush_l2("read")
        step()
    torch.cuda.synchronize()

    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    # the SM clock and the throttle reasons are sampled (NVML, every 0.5 ms) while the timed steps run and, further
    # down, while the hooked launches of the roofline object run: both are the load the reported numbers come from
    clocks = clk.ClockSampler(local, str(torch.cuda.get_device_properties(local).uuid), period_s=0.0005)
    with clocks:
        for k in range(K):
            flush_l2("read")                      # untimed: evicts X and the outputs from L2
            ev[k][0].record()
            step()
            ev[k][1].record()
        torch.cuda.synchronize()
    step_samples, step_reasons = list(clocks.samples), set(clocks.reasons)
    if world > 1:
        dist.barrier()
    step_ms = [e[0].elapsed_time(e[1]) for e in ev]
    total_ms = max_over_ranks(sum(step_ms), "cuda")
    value = whole_job_gbs(n, K, world, total_ms)
    zero_count = int(buf.zero_count.item())

    # ---- the dominant kernel (the quantize pass) timed inside real calls, outside the headline loop: the two extra
    # event records sit between dependent kernels and cost the call a few microseconds of overlap
    hook = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(HOOK_LAUNCHES)]
    for a_, b_ in hook:                              # torch creates the CUDA event on first record
        a_.record()
        b_.record()
    torch.cuda.synchronize()
    with clocks:
        for a_, b_ in hook:
            flush_l2("read")
            cq.set_timing_events(a_, b_)
            step()
        torch.cuda.synchronize()
    cq.set_timing_events(None, None)
    clocks.samples = step_samples + clocks.samples
    clocks.reasons |= step_reasons
    quant_ms = [a_.elapsed_time(b_) for a_, b_ in hook]

    # ---- end to end: host buffers in, host buffers out, through cq_quantize_act_host.
    # (a) one call after the other on one stream; (b) the same calls issued alternately on two streams with
    # their own buffers, so one step's download overlaps the next step's upload (PCIe is full duplex).
    Xp = Xh.pin_memory()
    hbs = [cq.HostBuffers(T, I, torch.bfloat16, BITS) for _ in range(E2E_STREAMS)]
    Ke = max(1, args.e2e_steps)
    for hb in hbs:
        cq.quantize_act_host(Xp, ALPHA, BITS, buffers=hb)
    torch.cuda.synchronize()
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(Ke)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(Ke)]
    if world > 1:
        dist.barrier()
    for k in range(Ke):
        e0[k].record()
        cq.quantize_act_host(Xp, ALPHA, BITS, buffers=hbs[0])
        e1[k].record()
    torch.cuda.synchronize()
    serial_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in zip(e0, e1)), "cuda")
    e2e_serial = whole_job_gbs(n, Ke, world, serial_ms)
    assert int(hbs[0].zero_count.item()) == zero_count

    streams = [torch.cuda.Stream() for _ in range(E2E_STREAMS)]
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    p0.record()
    for st in streams:
        st.wait_event(p0)
    for k in range(Ke):
        with torch.cuda.stream(streams[k % E2E_STREAMS]):
            cq.quantize_act_host(Xp, ALPHA, BITS, buffers=hbs[k % E2E_STREAMS])
    for st in streams:
        torch.cuda.current_stream().wait_stream(st)
    p1.record()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(p0.elapsed_time(p1), "cuda")
    e2e_value = whole_job_gbs(n, Ke, world, e2e_ms)
    assert all(int(hbs[k % E2E_STREAMS].zero_count.item()) == zero_count for k in range(min(Ke, E2E_STREAMS)))
    hb = hbs[0]

    # ---- also: INT4 codes on the same matrix and the per-channel weight quantizer (not part of `value`)
    def timed(fn, iters=40, flushed=True):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        for _ in range(3):
            fn()
        for a_, b_ in evs:
            if flushed:
                flush_l2(flushed if isinstance(flushed, str) else "read")
            a_.record()
            fn()
            b_.record()
        torch.cuda.synchronize()
        return statistics.median(a_.elapsed_time(b_) for a_, b_ in evs)
    also = {}
    if rank == 0:
        buf4 = cq.ActBuffers(T, I, torch.bfloat16, 4)
        ms4 = timed(lambda: cq.quantize_act(Xd, ALPHA, 4, buffers=buf4))
        also["act_int4"] = {"ms_per_step": ms4, "gbs": 6.5 * n / (ms4 * 1e-3) / 1e9, "bytes_per_element": 6.5}
        del buf4
        msw8 = timed(lambda: cq.quantize_act(Xd, ALPHA, BITS, buffers=buf), flushed="write")
        also["act_int8_after_a_write_flush"] = {
            "ms_per_step": msw8, "gbs": BYTES_PER_ELEMENT_STEP * n / (msw8 * 1e-3) / 1e9,
            "l2": "flushed by a 256 MiB fill: the write-back of its 126 MB of dirty lines overlaps the absmax pass"}
        ms8 = timed(lambda: cq.quantize_act(Xd, ALPHA, BITS, buffers=buf), flushed=False)
        also["act_int8_back_to_back"] = {"ms_per_step": ms8, "gbs": BYTES_PER_ELEMENT_STEP * n / (ms8 * 1e-3) / 1e9,
                                         "l2": "not flushed: X (235 MB) and the outputs (352 MB) exceed the 126 MB L2"}
        Wd = torch.from_numpy(wl.sweep_weight(0, 2).view(np.int16)).view(torch.bfloat16).cuda()
        wout = cq.quantize_weight_per_channel(Wd, 8)
        msw = timed(lambda: cq.quantize_weight_per_channel(Wd, 8, out=wout))
        also["weight_per_channel_int8_28672x8192"] = {"ms": msw, "gbs": 5.0 * Wd.numel() / (msw * 1e-3) / 1e9,
                                                       "bytes_per_element": 5.0}
        del Wd, wout

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    quant_mean_ms = statistics.fmean(quant_ms)
    achieved = BYTES_PER_ELEMENT_QUANT_PASS * n / (quant_mean_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC["bytes_per_launch"] if NCU_TRAFFIC["sources_sha256"] == kernel_sources_digest() else None

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(cfg),
                   "l2": "flushed between steps by reading a 256 MiB buffer twice, untimed (clean lines); X (235 MB) also exceeds the "
                         "126 MB L2; the same step after a 256 MiB write flush and back to back: see also",
                   "timing": "CUDA events per step on the launch stream, summed; max over ranks",
                   "bytes_per_element": BYTES_PER_ELEMENT_STEP, "per_rank": "independent matrices, no collective"},
        "elements_per_s": n * K * world / (total_ms * 1e-3),
        "fraction_of_hbm_roofline": value / (peak * world),
        "ms_per_step_median": statistics.median(step_ms),
        "kernel_proportion": zero_count / n,
        "clocks": clocks.summary(),
        "gpu_launches": 3 * K,
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": Ke,
                "h2d_bytes_per_step": X.nbytes, "d2h_bytes_per_step": hb.d2h_bytes(),
                "api": "cq_quantize_act_host (pinned host buffers; copies inside the timed region), calls issued "
                       "alternately on two streams so a step's download overlaps the next step's upload",
                "one_stream_value": e2e_serial},
        "also": also,
        "roofline": {"bound": "hbm", "kernel": "k3_quantize (quantize / pack / dequantize / zero-count pass)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": traffic,
                     "algorithmic_bytes_per_launch": BYTES_PER_ELEMENT_QUANT_PASS * n,
                     "avg_launch_ms": quant_mean_ms, "launches_timed": len(quant_ms)},
    }

    # ---- the oracle on the host cores, bounded sample of the same workload
    from oracle import cq_oracle as orc
    orc.quantize_act(X[:64], cfg.dtype, ALPHA, BITS, want_deq32=False)
    reps, t0 = 0, time.perf_counter()
    while reps < 3 or (time.perf_counter() - t0 < 1.5 and reps < 50):
        orc.quantize_act(X, cfg.dtype, ALPHA, BITS, want_deq32=False)
        reps += 1
    dt = time.perf_counter() - t0
    all_threads = orc.num_threads()
    Xs = np.ascontiguousarray(X[:256])                                   # one core: a 256-row sample is enough
    orc.set_num_threads(1)
    t1 = time.perf_counter()
    orc.quantize_act(Xs, cfg.dtype, ALPHA, BITS, want_deq32=False)
    dt1 = time.perf_counter() - t1
    orc.set_num_threads(all_threads)
    out["cpu_baseline"] = {"value": BYTES_PER_ELEMENT_STEP * X.size * reps / dt / 1e9, "unit": UNIT,
                           "cores": all_threads, "kind": "oracle",
                           "single_thread_value": BYTES_PER_ELEMENT_STEP * Xs.size / dt1 / 1e9,
                           "host_cores": os.cpu_count(),
                           "sample": f"the whole workload matrix ({T}x{I}), {reps} oracle quantize_act calls "
                                     f"(t, c, codes, bf16 dequant, count) in {dt:.2f} s wall on {orc.num_threads()} threads"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
