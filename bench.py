#!/usr/bin/env python
"""Benchmark of the DPPF consensus round (pull-push update, Sec. 5 of the paper).

One "step" is one consensus round over all M replicas of the workload: average,
per-worker distances, in-place pull-push update.  The default workload is the
ViT-B/16-sized one (M = 4, d = 86,567,656 fp32), one call of the library per round,
rounds issued back to back on one stream.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--workload C4]
                    [--variant plain|general|adamw] [--shard none|columns] [--impl ours|reference]

The K-step loop is timed R times (each time bracketed by a barrier and a device
synchronisation, CUDA events on the launching stream, slowest rank counts); the
reported time per step is the median over the R repeats.

--variant plain     dppf_consensus per step (workload C3: the last local SGD-momentum step fused
                    with the round, dppf_local_step_and_consensus); also reports, under
                    "multi_round", the same rounds issued 100 per call through
                    dppf_consensus_rounds (update pass of round k fused with the distance pass of
                    round k+1).
--variant general   dppf_consensus_general (weighted consensus variable, push from it, both terms).
--variant adamw     dppf_adamw_step_and_consensus (last AdamW step fused with the round).

Multi-GPU: by default the path does not shard (one GPU holds all M replicas of a round), so
N > 1 runs N independent replicas, one process per GPU, with no data-path collective ("weak"
scaling: rounds/s adds up).  --shard columns splits the columns of ONE workload over the N
ranks instead: every step is dppf_distance_partials, an all-reduce of the M fp64 sums of
squares, dppf_update_from_sums ("strong" scaling).  --shard workers is the paper's own
arrangement, one replica per GPU (needs N = M ranks): every step is an all-reduce (sum) of the
d parameters and dppf_worker_update; with N = 1 the all-reduce is left out and only the
worker kernel is timed.

``--impl reference`` times the CPU oracle (plain C, fp64) on the host cores on a
bounded column slice of the same workload; rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "DPPF consensus rounds/s"
UNIT = "rounds/s"
NOMINAL_HBM_GBS = 8000.0
ADAMW = dict(lr=5e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)     # the paper's ViT setting


def parse_args(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--repeats", type=int, default=20, help="how many times the K-step loop is timed (median reported)")
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="C4")
    p.add_argument("--variant", default="plain", choices=["plain", "general", "adamw"])
    p.add_argument("--shard", default="none", choices=["none", "columns", "workers"])
    p.add_argument("--d", type=int, default=0, help="override the vector length (profiling on a smaller case)")
    p.add_argument("--path", default="auto", choices=["auto", "two_kernel", "cooperative", "staged"])
    p.add_argument("--rounds-per-call", type=int, default=100, help="rounds per dppf_consensus_rounds call")
    p.add_argument("--multi-round-calls", type=int, default=7)
    p.add_argument("--no-multi-round", action="store_true")
    p.add_argument("--e2e-steps", type=int, default=5)
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--seed", type=int, default=None)
    p.add_argument("--graph", action="store_true",
                   help="also time the same steps replayed from a CUDA graph (extra key 'graph_replay')")
    return p.parse_args(argv)


def measured_peaks():
    """(hbm GB/s, source): the measured copy bandwidth of this machine's B200s, else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from single-pass ncu
# captures of full-size launches.  Keyed by (workload, d, kernel); an entry is removed whenever
# that kernel changes, and the line then reports null.
NCU_TRAFFIC = {
    ("C4", 86_567_656, "round_kernel_staged"): 4.008e9,
    ("C4", 86_567_656, "rounds100"): 264.5e9,
    ("C2", 26_200_000, "round_kernel_staged"): 2.369e9,
    ("C5", 44_549_160, "rounds_kernel_staged"): 8.411e9,
    ("C3", 25_557_032, "fused_round_kernel_staged"): 2.746e9,
    ("C4", 86_567_656, "general_round_kernel"): 4.004e9,
    ("C4", 86_567_656, "adamw_round_kernel"): 12.365e9,
    ("C4", 86_567_656, "worker_round_kernel"): 1.583e9,
}


def workload_of(args):
    from paper_2507_20424_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.d:
        w = w.scaled(args.d)
    return w


def step_description(w, variant):
    if variant == "general":
        return "general rounds (weighted consensus variable, push from it, both gradient terms)"
    if variant == "adamw":
        return "last AdamW local step fused with the round, steps"
    return "last local SGD-momentum step fused with the round, steps" if w.tau > 0 else "rounds"


def config_of(w, variant="plain"):
    """Names the workload; identical in the CUDA arm and the reference arm."""
    return {"workload": f"{w.name}: M={w.M} replicas x d={w.d} fp32 ({w.model}), alpha={w.alpha}, lambda={w.lam}, "
                        f"{step_description(w, variant)} back to back on one stream",
            "variant": variant, "M": w.M, "d": w.d, "ld": w.ld, "alpha": w.alpha, "lambda": w.lam,
            "replica_bytes": w.M * w.d * 4,
            "l2_policy": "inputs larger than L2 (no flush between iterations)"}


def general_weights(w, seed):
    """Seeded positive weights of the consensus variable for --variant general."""
    import numpy as np
    return (np.random.default_rng(seed).random(w.M) + 0.05).astype(np.float32)


def column_shard(d, world, rank):
    """Columns [lo, hi) of rank `rank` when d columns are split over `world` ranks: equal
    shares rounded up to 32 columns (128-byte row starts), the last rank takes the rest."""
    per = -(-d // world)
    per = -(-per // 32) * 32
    lo = min(d, rank * per)
    hi = d if rank == world - 1 else min(d, lo + per)
    return lo, hi


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, period=0.005):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self.period = period
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.reason_bits |= int(get(self.h))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
            try:                      # one more sample while the last launches drain
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            except Exception:
                pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "samples": len(s),
                "reasons": [name for bit, name in self.REASONS.items() if self.reason_bits & bit]}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ------------------------------------------------------------------ CPU oracle legs

def _with_grad_std(w):
    from dataclasses import replace
    return replace(w, grad_std=1e-2)


def oracle_step_fn(w, variant, seed, d_s):
    """Returns (one_step, cores): one_step() runs one oracle step of the variant on the first
    d_s columns of the workload, carrying its state from call to call."""
    import numpy as np
    import oracle
    from paper_2507_20424_b200 import inputs
    ws = w.scaled(d_s)
    x0 = np.ascontiguousarray(inputs.replicas(ws, seed)[:, :d_s])
    if variant == "general":
        wts = general_weights(w, seed)
        state = {"x": x0}

        def one_step():
            state["x"], _, _ = oracle.consensus_general(state["x"], w.alpha, w.lam, wts, "consensus", True, d=d_s)
        return one_step, 1
    if variant == "adamw":
        g = np.ascontiguousarray(inputs.gradients(ws if ws.grad_std else _with_grad_std(ws), 0, seed)[:, :d_s])
        state = {"x": x0.astype(np.float64), "a": np.zeros((w.M, d_s)), "b": np.zeros((w.M, d_s)), "t": 0}

        def one_step():
            state["t"] += 1
            x64, state["a"], state["b"] = oracle.adamw_steps_f64(state["x"], state["a"], state["b"], [g],
                                                                first_step=state["t"], **ADAMW)
            out, _ = oracle.consensus_f64(x64, w.alpha, w.lam)
            state["x"] = out.astype(np.float64)
        return one_step, 1
    if w.tau > 0:          # local-step workload: one oracle local step, then the round, per step
        g = np.ascontiguousarray(inputs.gradients(ws, 0, seed)[:, :d_s])
        state = {"x": x0, "v": np.zeros((w.M, d_s), dtype=np.float32)}

        def one_step():
            xo, v64, _ = oracle.local_steps_then_consensus(state["x"], state["v"], [g], w.lr, w.momentum,
                                                           w.weight_decay, w.alpha, w.lam)
            state["x"], state["v"] = xo, v64.astype(np.float32)
        return one_step, 1
    state = {"x": x0, "cores": 0}

    def one_step():
        state["x"], _, state["cores"] = oracle.consensus_blocked(state["x"], w.alpha, w.lam, d=d_s)
    one_step()
    return one_step, state["cores"]


def time_oracle(w, variant, seed, budget_s):
    """Times one oracle step of the variant on a column slice sized for about ``budget_s``
    seconds; returns (full-workload rounds/s, threads used, slice, seconds)."""
    import oracle
    oracle.build()
    probe = min(w.d, 1_000_000)
    step, cores = oracle_step_fn(w, variant, seed, probe)
    t0 = time.perf_counter()
    step()
    rate = probe / max(time.perf_counter() - t0, 1e-6)          # columns per second
    d_s = int(min(w.d, max(probe, rate * budget_s)))
    step, cores = oracle_step_fn(w, variant, seed, d_s)
    reps = int(min(50, max(1, budget_s * rate / d_s)))          # whole workload within the budget: repeat it
    t0 = time.perf_counter()
    for _ in range(reps):
        step()
    dt = (time.perf_counter() - t0) / reps
    return 1.0 / (dt * w.d / d_s), cores, d_s, dt * reps


def single_thread_oracle_rate(w, seed, budget_s):
    """Full-workload rounds/s of the oracle's round on ONE thread, from a column slice."""
    import numpy as np
    import oracle
    from paper_2507_20424_b200 import inputs
    probe = min(w.d, 500_000)
    x = np.ascontiguousarray(inputs.replicas(w.scaled(probe), seed)[:, :probe])
    t0 = time.perf_counter()
    oracle.consensus_blocked(x, w.alpha, w.lam, d=probe, threads=1)
    rate = probe / max(time.perf_counter() - t0, 1e-6)
    d_s = int(min(w.d, max(probe, rate * budget_s)))
    x = np.ascontiguousarray(inputs.replicas(w.scaled(d_s), seed)[:, :d_s])
    t0 = time.perf_counter()
    oracle.consensus_blocked(x, w.alpha, w.lam, d=d_s, threads=1)
    return 1.0 / ((time.perf_counter() - t0) * w.d / d_s)


def run_reference(args):
    """The CPU oracle as the reference arm: rank 0 only, bounded column slice per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2507_20424_b200 import inputs
    oracle.build()
    w = workload_of(args)
    seed = inputs.DEFAULT_SEED if args.seed is None else args.seed
    total_budget = 150.0
    per_step = total_budget / max(1, args.steps + args.warmup)
    # calibrate on a small slice, then size the per-step slice
    probe = min(w.d, 500_000)
    step, cores = oracle_step_fn(w, args.variant, seed, probe)
    t0 = time.perf_counter()
    step()
    rate = probe / max(time.perf_counter() - t0, 1e-6)
    d_s = int(min(w.d, max(4096, rate * per_step * 0.8)))
    one_step, cores = oracle_step_fn(w, args.variant, seed, d_s)
    for _ in range(args.warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = 1.0 / (dt * w.d / d_s)
    what = {"general": "one oracle general round", "adamw": "one oracle AdamW step and round"}.get(
        args.variant, "one oracle local step and round" if w.tau > 0 else "one oracle round")
    sample = (f"each step = {what} on the first {d_s} of {w.d} columns (all {w.M} rows); "
              f"rounds/s scaled by {d_s}/{w.d}")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * w.d / d_s * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(w, args.variant),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ aggregation over ranks

def max_over_ranks(ms, world, device=None):
    """Slowest rank's elapsed time: the job is done when the last rank is."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(steps, world, elapsed_ms):
    """Rounds per second over all ranks: every rank ran `steps` rounds on its own replica set."""
    return world * steps / (elapsed_ms * 1e-3)


# ------------------------------------------------------------------ CUDA arm

def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2507_20424_b200 import binding, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    binding.load(rebuild_if_stale=True)
    w = workload_of(args)
    sharded = args.shard == "columns"
    per_worker = args.shard == "workers"
    variant = args.variant
    if (sharded or per_worker) and (variant != "plain" or w.tau > 0):
        raise SystemExit("--shard applies to the plain round")
    if per_worker and world not in (1, w.M):
        raise SystemExit(f"--shard workers needs one rank per worker ({w.M}) or a single rank")
    # replicas-only runs give every rank its own replica set; column shards share one
    seed = (inputs.DEFAULT_SEED if args.seed is None else args.seed) + (0 if (sharded or per_worker) else rank)
    path = {"auto": binding.PATH_AUTO, "two_kernel": binding.PATH_TWO_KERNEL,
            "cooperative": binding.PATH_COOPERATIVE, "staged": binding.PATH_STAGED}[args.path]

    # CPU baseline first (rank 0, N = 1 only): before any GPU work, so the OpenMP team is
    # created in a process that has not touched CUDA yet.
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, cores, d_s, dt = time_oracle(w, variant, seed, budget_s=12.0)
        cpu = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"oracle steps on the first {d_s} of {w.d} columns for {dt:.1f} s, rate scaled by columns"}
        if variant == "plain" and w.tau == 0:      # the same oracle on one thread, on a shorter slice
            cpu["single_thread_value"] = single_thread_oracle_rate(w, seed, budget_s=5.0)

    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    x_host = inputs.replicas(w, seed)
    lo, hi = column_shard(w.d, world, rank) if sharded else (0, w.d)
    d_loc = hi - lo
    x_pinned = torch.from_numpy(np.ascontiguousarray(x_host[:, lo:hi]) if sharded else x_host).pin_memory()
    x = binding.alloc_rows(w.M, d_loc)
    x[:, :d_loc].copy_(x_pinned[:, :d_loc], non_blocking=True)
    norms = torch.zeros(w.M, device="cuda")
    ws = binding.alloc_workspace(w.M, d_loc)
    B = w.M * d_loc * 4                      # replica bytes this rank holds
    fused_sgd = variant == "plain" and w.tau > 0
    staged = args.path in ("auto", "staged") and w.M <= 16

    if per_worker:
        # this rank's replica as a flat vector; the reduced vector is what a sum all-reduce leaves
        xw = torch.from_numpy(np.ascontiguousarray(x_host[rank, :w.d])).cuda()
        red = torch.from_numpy(np.ascontiguousarray(x_host[:, :w.d].astype(np.float64).sum(axis=0)
                                                    .astype(np.float32))).cuda()
        ws = binding.alloc_workspace(1, w.d)
        norms = torch.zeros(1, device="cuda")
        B = w.d * 4
        model_units, kernel_id = 5.0, "worker_round_kernel"
        kernel_name = ("all-reduce (sum) of the d parameters, then worker_round_kernel (distance pass, grid barrier, "
                       "update pass on this worker's replica)" if world > 1 else
                       "worker_round_kernel (distance pass, grid barrier, update pass on one replica; the all-reduce "
                       "is left out on a single GPU)")
        launches_per_step = 1

        def step():
            if world > 1:
                red.copy_(xw)
                dist.all_reduce(red)
            binding.dppf_worker_update(xw, red, 1.0 / w.M, w.alpha, w.lam, norm_out=norms, ws=ws)
    elif sharded:
        sums = torch.zeros(w.M, dtype=torch.float64, device="cuda")
        model_units, kernel_id = 3.0, "distance_kernel + update_kernel (column shard)"
        kernel_name = ("dppf_distance_partials (distance_kernel + sum_partials_kernel), all-reduce of M fp64 sums, "
                       "dppf_update_from_sums (update_kernel)")
        launches_per_step = 3

        def step():
            binding.dppf_distance_partials(x, sums, ws=ws, d=d_loc)
            if world > 1:
                dist.all_reduce(sums)
            binding.dppf_update_from_sums(x, w.alpha, w.lam, sums, norms_out=norms, d=d_loc)
    elif variant == "general":
        wts = [float(v) for v in general_weights(w, seed)]
        model_units, kernel_id = 3.0, "general_round_kernel"
        kernel_name = "general_round_kernel (distance pass + grid barrier + update pass, one launch)"
        launches_per_step = 1

        def step():
            binding.dppf_consensus_general(x, w.alpha, w.lam, wts, binding.PUSH_FROM_CONSENSUS, True,
                                           norms_out=norms, ws=ws, d=w.d)
    elif variant == "adamw":
        wg = w if w.grad_std else _with_grad_std(w)
        m1, m2 = binding.alloc_rows(w.M, w.d, fill=0.0), binding.alloc_rows(w.M, w.d, fill=0.0)
        g = binding.alloc_rows(w.M, w.d)
        g.copy_(torch.from_numpy(inputs.gradients(wg, 0, seed)).pin_memory(), non_blocking=True)
        model_units, kernel_id = 9.0, "adamw_round_kernel"
        kernel_name = "adamw_round_kernel (AdamW step + distance pass, grid barrier, update pass, one launch)"
        launches_per_step = binding.adamw_launch_count(w.M)
        counter = {"t": 0}

        def step():
            counter["t"] += 1
            binding.dppf_adamw_step_and_consensus(x, m1, m2, g, step=counter["t"], alpha=w.alpha, lam=w.lam,
                                                  norms_out=norms, ws=ws, d=w.d, **ADAMW)
    elif fused_sgd:
        v = binding.alloc_rows(w.M, w.d, fill=0.0)
        g = binding.alloc_rows(w.M, w.d)
        g.copy_(torch.from_numpy(inputs.gradients(w, 0, seed)).pin_memory(), non_blocking=True)
        model_units = 7.0                                          # two-pass fused round: 7 x M d 4 bytes
        kernel_id = ("two_kernel<fused>" if args.path == "two_kernel" else
                     "fused_round_kernel_staged" if staged and w.M <= 8 else "round_kernel<fused>")
        kernel_name = {"two_kernel<fused>": "distance_kernel<fused> + update_kernel (one step)",
                       "fused_round_kernel_staged": "fused_round_kernel_staged (local step + distance pass staged through "
                                                    "shared memory, grid barrier, staged update pass, one launch)",
                       "round_kernel<fused>": "round_kernel<fused> (local step + distance pass, grid barrier, update "
                                              "pass, one launch)"}[kernel_id]
        launches_per_step = binding.launch_count(w.M, w.d, path, True)

        def step():
            binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay, w.alpha, w.lam,
                                                  norms_out=norms, ws=ws, d=w.d, path=path)
    else:
        model_units = 3.0
        kernel_id = ("two_kernel" if args.path == "two_kernel" else "round_kernel_staged" if staged and w.M <= 8 else
                     "rounds_kernel_staged" if staged else "round_kernel")
        kernel_name = {"two_kernel": "distance_kernel + update_kernel (one round)",
                       "round_kernel_staged": "round_kernel_staged (distance pass + grid barrier + update pass, one launch)",
                       "rounds_kernel_staged": "rounds_kernel_staged, one round (distance pass + grid barrier + update pass, one launch)",
                       "round_kernel": "round_kernel (distance pass + grid barrier + update pass, one launch)"}[kernel_id]
        launches_per_step = binding.launch_count(w.M, w.d, path, False)

        def step():
            binding.dppf_consensus(x, w.alpha, w.lam, norms_out=norms, ws=ws, d=w.d, path=path)

    def fence():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    fence()
    K, R = args.steps, max(1, args.repeats)
    rep_ms, launch_ms = [], []
    with ClockSampler(physical_gpu_index(local)) as clocks:
        for _ in range(R):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
            fence()
            ev[0].record()
            for i in range(K):
                step()
                ev[i + 1].record()
            fence()
            rep_ms.append(max_over_ranks(ev[0].elapsed_time(ev[K]), world, "cuda"))
            launch_ms.append(sum(ev[i].elapsed_time(ev[i + 1]) for i in range(K)) / K)
    if binding.dppf_device_status(ws) != binding.OK:
        raise SystemExit("device status word reports an error")
    total_ms = statistics.median(rep_ms)
    per_launch_ms = statistics.median(launch_ms)
    peak, peak_src = measured_peaks()

    # the same rounds, rounds_per_call of them per library call (update pass of round k fused with
    # the distance pass of round k + 1): (1 + 2n) x M d 4 bytes per call
    multi_round = None
    if variant == "plain" and not fused_sgd and not sharded and not per_worker and not args.no_multi_round and w.M <= 16:
        n = args.rounds_per_call
        norms_all = torch.zeros(n, w.M, device="cuda")
        binding.dppf_consensus_rounds(x, w.alpha, w.lam, n, norms_out=norms_all, ws=ws, d=w.d)
        fence()
        call_ms = []
        for _ in range(max(1, args.multi_round_calls)):
            m0, m1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fence()
            m0.record()
            binding.dppf_consensus_rounds(x, w.alpha, w.lam, n, norms_out=norms_all, ws=ws, d=w.d)
            m1_.record()
            fence()
            call_ms.append(max_over_ranks(m0.elapsed_time(m1_), world, "cuda"))
        if binding.dppf_device_status(ws) != binding.OK:
            raise SystemExit("device status word reports an error")
        ms = statistics.median(call_ms)
        alg = (1 + 2 * n) * B
        multi_round = {"entry": "dppf_consensus_rounds", "rounds_per_call": n, "calls_timed": len(call_ms),
                       "value": whole_job_rate(n, world, ms), "unit": UNIT, "ms_per_round": ms / n,
                       "ms_per_call_min_max": [min(call_ms), max(call_ms)],
                       "algorithmic_bytes_per_call": alg, "achieved": alg / (ms * 1e-3) / 1e9, "peak": peak,
                       "frac": alg / (ms * 1e-3) / 1e9 / peak, "traffic": NCU_TRAFFIC.get((w.name, w.d, f"rounds{n}")),
                       "kernel": "rounds_kernel_staged (distance pass, then per round: grid barrier + update pass "
                                 "that also accumulates the next round's squared distances; one launch)",
                       "gpu_launches_per_call": 1, "model_3Md4_equivalent_gbs": 3 * n * B / (ms * 1e-3) / 1e9}

    # optional: the same K steps captured once into a CUDA graph and replayed (launch overhead off the host)
    graph_replay = None
    if args.graph and not sharded and not per_worker and variant != "adamw":
        chunk = min(K, 100)
        cg_ = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg_):
            for _ in range(chunk):
                step()
        reps = max(1, K // chunk)
        cg_.replay()
        fence()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(reps):
            cg_.replay()
        g1.record()
        fence()
        g_ms = max_over_ranks(g0.elapsed_time(g1), world, "cuda")
        graph_replay = {"value": whole_job_rate(reps * chunk, world, g_ms), "unit": UNIT,
                        "steps_per_graph": chunk, "replays": reps, "ms_per_step": g_ms / (reps * chunk)}

    # end-to-end: replicas live in pinned host memory; every step copies them in, runs the
    # round and copies the replicas and the M distances back.
    e2e = None
    if not args.no_e2e and variant == "plain" and not fused_sgd and not sharded and not per_worker:
        norms_host = torch.zeros(w.M).pin_memory()
        binding.dppf_consensus_host(x_pinned, w.alpha, w.lam, norms_host, x, ws, d=w.d)
        fence()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            binding.dppf_consensus_host(x_pinned, w.alpha, w.lam, norms_host, x, ws, d=w.d)
        e1.record()
        fence()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        e2e = {"value": whole_job_rate(args.e2e_steps, world, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": B, "d2h_bytes_per_step": B + 4 * w.M, "steps": args.e2e_steps}

    if rank == 0:
        jobs = 1 if (sharded or per_worker) else world   # shards: all ranks work on ONE round
        achieved = model_units * B / (per_launch_ms * 1e-3) / 1e9
        value = whole_job_rate(K, jobs, total_ms)
        model_gbs = model_units * B * K / (total_ms * 1e-3) / 1e9
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                "warmup": max(3, args.warmup), "repeats": R, "ms_per_step": total_ms / K,
                "ms_per_step_min_max": [min(rep_ms) / K, max(rep_ms) / K],
                "higher_is_better": True, "scaling": "strong" if (sharded or per_worker) else "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic", "config": config_of(w, variant),
                "parallelism": (f"one replica per GPU x{world} (all-reduce of d fp32 per round)" if per_worker and world > 1
                                else "one replica of the workload on one GPU (no all-reduce)" if per_worker else
                                f"column shards x{world} (all-reduce of {w.M} fp64 sums per round)" if sharded else
                                f"replicas x{world}" if world > 1 else "single GPU"),
                "schedule": args.path,
                "model_gbs_per_gpu": model_gbs, "frac_of_nominal_8tbs": model_gbs / NOMINAL_HBM_GBS,
                "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "traffic": NCU_TRAFFIC.get((w.name, w.d, kernel_id)),
                             "kernel": kernel_name,
                             "algorithmic_bytes_per_launch": int(model_units) * B, "peak_source": f"of {peak_src}"},
                "clocks": clocks.summary(), "gpu_launches": R * K * launches_per_step,
                "norms_last_round": [float(v) for v in norms.cpu().tolist()]}
        if multi_round is not None:
            line["multi_round"] = multi_round
        if graph_replay is not None:
            line["graph_replay"] = graph_replay
        if e2e is not None:
            line["e2e"] = e2e
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
