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


# ---- one matrix split by rows over two ranks: the exchange step (column maxima MAX, kernel sizes SUM) ----
SHARD_WORKER = r"""
import json, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_2410_07505_b200 import sharded, workloads as wl
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
X = wl.bits_to_f32(wl.small_matrix(37, 24, wl.BF16, 11), wl.BF16)          # the same matrix on both ranks
r0, r1 = sharded.shard_rows(37, 2, rank)
c_local = torch.from_numpy(np.abs(X[r0:r1]).max(axis=0).astype(np.float32))    # stands in for the absmax kernel
c = sharded.combine_column_maxima(c_local.clone())
total = sharded.combine_counts(torch.tensor(100 + rank, dtype=torch.int64))
print(json.dumps({{"rank": rank, "rows": [r0, r1], "c": c.tolist(), "c_full": np.abs(X).max(axis=0).tolist(),
                  "total": int(total)}}))
dist.barrier()
dist.destroy_process_group()
"""


def test_row_shards_exchange_column_maxima_and_counts(tmp_path):
    port = 31500 + os.getpid() % 2000
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True, cwd=ROOT) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["rows"] == [0, 19] and outs[1]["rows"] == [19, 37]          # contiguous, sizes differ by one
    for o in outs:
        assert o["c"] == o["c_full"]                                            # every rank ends with the global maxima
        assert o["total"] == 201                                                # and with the sum of the counts


def test_shard_rows_partition():
    from paper_2410_07505_b200 import sharded
    for T in (0, 1, 7, 4096):
        for world in (1, 2, 3, 8):
            spans = [sharded.shard_rows(T, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


# ---- bench.py --gpus N run directly starts its own N ranks (checked on the CPU through --dry-run) ----
def test_bench_starts_its_own_ranks_and_never_runs_with_fewer():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env,
                       capture_output=True, text=True, cwd=ROOT, timeout=600)
    assert p.returncode == 0, p.stderr[-3000:]
    line = json.loads([ln for ln in p.stdout.strip().splitlines() if ln.startswith("{")][-1])
    assert line["dry_run"] and line["n_gpus"] == 2 and line["ranks_seen"] == 2
    assert line["max_ms"] == 2.0 and len(set(line["seeds"])) == 2
    # a launcher's world size that disagrees with --gpus is an error, not a quiet single-rank run
    env_bad = dict(env, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env_bad,
                       capture_output=True, text=True, cwd=ROOT, timeout=120)
    assert p.returncode != 0 and "WORLD_SIZE" in p.stderr
    # more ranks than visible GPUs (none here) is refused before anything is started
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], env=dict(env, CUDA_VISIBLE_DEVICES=""),
                       capture_output=True, text=True, cwd=ROOT, timeout=120)
    assert p.returncode != 0 and "refusing" in p.stderr
