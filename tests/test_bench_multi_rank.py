"""Host logic of the multi-GPU benchmark arm ("replicas only": N independent copies of the
workload, no data-path collective), run as two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
import bench
from paper_2507_20424_b200 import inputs
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# every rank draws its own replica set (seed + rank), as the CUDA arm does
w = inputs.WORKLOADS["C1"].scaled(1000)
x = inputs.replicas(w, inputs.DEFAULT_SEED + rank)
checksum = float(x[:, :w.d].astype("float64").sum())
sums = [None] * world
dist.all_gather_object(sums, checksum)
# rank r pretends its timed region took (10 + 5 r) ms for 100 rounds
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)
rate = bench.whole_job_rate(100, world, ms)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "rate": rate, "distinct_inputs": len(set(sums)) == world}))
dist.destroy_process_group()
"""


def test_two_ranks_report_slowest_time_and_summed_rate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script), ROOT]
    run = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert run.returncode == 0, run.stderr[-2000:]
    line = [l for l in run.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["ms"] == 15.0                                   # the slower rank
    assert out["rate"] == pytest.approx(2 * 100 / 0.015)       # both replicas' rounds count
    assert out["distinct_inputs"]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, 1) == 12.5
    assert bench.whole_job_rate(1000, 1, 500.0) == 2000.0


def test_reference_arm_prints_one_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert run.returncode == 0 and run.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--workload", "C1", "--gpus", "2"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert run.returncode == 0, run.stderr[-2000:]
    lines = [l for l in run.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["unit"] == "rounds/s" and out["value"] > 0
    assert out["cpu_baseline"]["kind"] == "oracle" and out["cpu_baseline"]["cores"] >= 1
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["e2e"]["d2h_bytes_per_step"] == 0


SHARD_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np
import torch, torch.distributed as dist
import bench, oracle
from paper_2507_20424_b200 import inputs
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# column shards of ONE replica set (same seed on every rank)
w = inputs.WORKLOADS["C1"].scaled(10_007)
x = inputs.replicas(w)
lo, hi = bench.column_shard(w.d, world, rank)
# this rank's share of the sums of squares: the oracle's distances on its own columns, squared
_, r_shard = oracle.consensus(np.ascontiguousarray(x[:, lo:hi]), w.alpha, 0.0)
sums = torch.from_numpy(r_shard ** 2)
dist.all_reduce(sums)                                   # the one exchange of a column-sharded round
spans = [None] * world
dist.all_gather_object(spans, (lo, hi))
_, r_full = oracle.consensus(x, w.alpha, 0.0, d=w.d)
if rank == 0:
    print(json.dumps({"spans": spans, "d": w.d, "r": np.sqrt(sums.numpy()).tolist(), "r_full": r_full.tolist()}))
dist.destroy_process_group()
"""


def test_two_ranks_column_shards_and_sum_exchange(tmp_path):
    """Column shards tile [0, d) on 128-byte boundaries, and adding the shards' sums of squares
    over the ranks gives the distances of the whole vector."""
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29534", str(script), ROOT]
    run = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert run.returncode == 0, run.stderr[-2000:]
    out = json.loads([l for l in run.stdout.splitlines() if l.startswith("{")][-1])
    (lo0, hi0), (lo1, hi1) = out["spans"]
    assert lo0 == 0 and hi0 == lo1 and hi1 == out["d"] and lo1 % 32 == 0
    assert out["r"] == pytest.approx(out["r_full"], rel=1e-12)


def test_column_shard_covers_every_column_once():
    sys.path.insert(0, ROOT)
    import bench
    for d in (1, 31, 32, 33, 1000, 86_567_656):
        for world in (1, 2, 3, 8):
            spans = [bench.column_shard(d, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == d
            for (lo, hi), (lo2, _) in zip(spans[:-1], spans[1:]):
                assert hi == lo2 and lo <= hi
            assert all(lo % 32 == 0 or lo == hi for lo, hi in spans)      # non-empty shards start on 128 bytes


WORKER_PER_RANK = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np
import torch, torch.distributed as dist
import oracle
from paper_2507_20424_b200 import inputs
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# the paper's arrangement: rank m holds replica m; one all-reduce (sum) of the parameters per round
w = inputs.WORKLOADS["C1"].scaled(5003)
x_all = inputs.replicas(w)[:world, :w.d]                 # every rank could draw all, but uses only its own
mine = np.ascontiguousarray(x_all[rank])
reduced = torch.from_numpy(mine.copy())
dist.all_reduce(reduced)                                 # the one collective of the round
out, r = oracle.worker_update(mine, reduced.numpy(), 1.0 / world, w.alpha, w.lam)
ref, r_ref = oracle.consensus(np.ascontiguousarray(x_all), w.alpha, w.lam)
ok = bool(abs(r - r_ref[rank]) <= 1e-6 * r_ref[rank] and np.abs(out.astype(np.float64) - ref[rank]).max() <= 2e-8)
oks = [None] * world
dist.all_gather_object(oks, ok)
if rank == 0:
    print(json.dumps({"ok": oks}))
dist.destroy_process_group()
"""


def test_two_ranks_one_replica_each(tmp_path):
    """Rank m holds replica m, the parameters are all-reduced once, and each rank's own update
    (the oracle's one-worker form) reproduces its row of the oracle's round on both replicas."""
    script = tmp_path / "worker_per_rank.py"
    script.write_text(WORKER_PER_RANK)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29535", str(script), ROOT]
    run = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert run.returncode == 0, run.stderr[-2000:]
    out = json.loads([l for l in run.stdout.splitlines() if l.startswith("{")][-1])
    assert out["ok"] == [True, True]
