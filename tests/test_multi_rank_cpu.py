"""Host logic of the multi-GPU benchmark path, run as two gloo ranks on the CPU: independent
per-rank workloads (no data-path collective), max-over-ranks timing, whole-job aggregation."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys, dataclasses
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
from paper_2410_07505_b200 import workloads as wl
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
cfg = dataclasses.replace(bench.rank_config(rank), T=8, I=64)
X = wl.generate_activation(cfg)
local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
mx = bench.max_over_ranks(local_ms, "cpu")
value = bench.whole_job_gbs(1000, 4, 2, mx)
print(json.dumps({{"rank": rank, "seed": cfg.seed, "sum": int(X.sum(dtype="int64")), "max_ms": mx, "value": value}}))
dist.barrier()
dist.destroy_process_group()
"""


def test_two_gloo_ranks_aggregate_by_the_slowest(tmp_path):
    port = 29500 + os.getpid() % 2000
    script = tmp_path / "worker.py"
    script.write_text("import numpy as np\n" + WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True, cwd=ROOT) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["seed"] != outs[1]["seed"] and outs[0]["sum"] != outs[1]["sum"]      # independent inputs
    assert outs[0]["max_ms"] == outs[1]["max_ms"] == 15.0                                # the slowest rank's time
    want = 7.0 * 1000 * 4 * 2 / 15e-3 / 1e9
    assert outs[0]["value"] == pytest.approx(want) and outs[1]["value"] == pytest.approx(want)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, cwd=ROOT)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
