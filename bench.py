#!/usr/bin/env python
"""Benchmark of the DPPF consensus round (pull-push update, Sec. 5 of the paper).

One "step" is one consensus round over all M replicas of the workload: average,
per-worker distances, in-place pull-push update.  The default workload is the
ViT-B/16-sized one (M = 4, d = 86,567,656 fp32), rounds issued back to back on one
stream.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4] [--impl ours|reference]

Multi-GPU: the path does not shard (one GPU holds all M replicas of a round), so
N > 1 runs N independent replicas, one process per GPU, with no data-path
collective ("weak" scaling: rounds/s adds up).

``--impl reference`` times the CPU oracle (plain C, fp64) on the host cores on a
bounded column slice of the same workload; rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "DPPF consensus rounds/s"
UNIT = "rounds/s"
NOMINAL_HBM_GBS = 8000.0


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=1000)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="C4")
    p.add_argument("--d", type=int, default=0, help="override the vector length (profiling on a smaller case)")
    p.add_argument("--path", default="auto", choices=["auto", "two_kernel", "cooperative", "staged"])
    p.add_argument("--e2e-steps", type=int, default=5)
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--seed", type=int, default=None)
    p.add_argument("--graph", action="store_true",
                   help="also time the same steps replayed from a CUDA graph (extra key 'graph_replay')")
    return p.parse_args()


def measured_peaks():
    """(hbm GB/s, source): the measured copy bandwidth of this machine's B200s, else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the single-pass
# ncu capture of the full-size launch summarised in profiles/round_kernel_staged_M4.md.
# Keyed by (workload, kernel); set an entry to None whenever that kernel changes.
NCU_TRAFFIC = {("C4", 86_567_656, "staged"): 4.00e9}


def measured_traffic(w, staged):
    return NCU_TRAFFIC.get((w.name, w.d, "staged" if staged else "register"))


def workload_of(args):
    from paper_2507_20424_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.d:
        w = w.scaled(args.d)
    return w


def config_of(w, extra=None):
    what = ("last local SGD-momentum step fused with the round, steps" if w.tau > 0 else "rounds")
    cfg = {"workload": f"{w.name}: M={w.M} replicas x d={w.d} fp32 ({w.model}), alpha={w.alpha}, lambda={w.lam}, "
                       f"{what} back to back on one stream",
           "M": w.M, "d": w.d, "ld": w.ld, "alpha": w.alpha, "lambda": w.lam,
           "replica_bytes": w.M * w.d * 4,
           "l2_policy": "inputs larger than L2 (no flush between iterations)"}
    if extra:
        cfg.update(extra)
    return cfg


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

def time_oracle(w, x_host, budget_s, threads=0):
    """Times the CPU oracle (column-block OpenMP variant) on a column slice sized for
    ``budget_s`` seconds; returns (full-workload rounds/s, threads used, slice, seconds)."""
    import oracle
    oracle.build()
    probe = min(w.d, 2_000_000)
    t0 = time.perf_counter()
    _, _, used = oracle.consensus_blocked(x_host[:, :probe], w.alpha, w.lam, threads=threads)
    rate = probe / max(time.perf_counter() - t0, 1e-6)          # columns per second
    d_s = int(min(w.d, max(probe, rate * budget_s)))
    t0 = time.perf_counter()
    oracle.consensus_blocked(x_host[:, :d_s], w.alpha, w.lam, threads=threads)
    dt = time.perf_counter() - t0
    return 1.0 / (dt * w.d / d_s), used, d_s, dt


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
    probe_w = w.scaled(min(w.d, 1_000_000))
    xp = inputs.replicas(probe_w, seed)
    t0 = time.perf_counter()
    _, _, cores = oracle.consensus_blocked(xp, w.alpha, w.lam, d=probe_w.d)
    rate = probe_w.d / max(time.perf_counter() - t0, 1e-6)
    d_s = int(min(w.d, max(4096, rate * per_step * 0.8)))
    fused = w.tau > 0          # local-step workload: one oracle local step, then the round, per step
    if fused:
        d_s = max(4096, d_s // 8)          # the oracle's local step is single-threaded fp64
        cores = 1
    ws = w.scaled(d_s)
    state = {"x": inputs.replicas(ws, seed)}
    if fused:
        import numpy as np
        g = np.ascontiguousarray(inputs.gradients(ws, 0, seed)[:, :d_s])
        state = {"x": np.ascontiguousarray(state["x"][:, :d_s]), "v": np.zeros((w.M, d_s), dtype=np.float32)}

        def one_step():
            xo, v64, _ = oracle.local_steps_then_consensus(state["x"], state["v"], [g], w.lr, w.momentum,
                                                           w.weight_decay, w.alpha, w.lam)
            state["x"], state["v"] = xo, v64.astype(np.float32)
    else:
        def one_step():
            state["x"], _, _ = oracle.consensus_blocked(state["x"], w.alpha, w.lam, d=d_s)
    for _ in range(args.warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = 1.0 / (dt * w.d / d_s)
    what = "one oracle local step and round" if fused else "one oracle round"
    sample = (f"each step = {what} on the first {d_s} of {w.d} columns (all {w.M} rows); "
              f"rounds/s scaled by {d_s}/{w.d}")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * w.d / d_s * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(w),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ replicas-only aggregation

def max_over_ranks(ms, world, device=None):
    """Slowest rank's elapsed time: the job is done when the last replica is."""
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
    seed = (inputs.DEFAULT_SEED if args.seed is None else args.seed) + rank
    path = {"auto": binding.PATH_AUTO, "two_kernel": binding.PATH_TWO_KERNEL,
            "cooperative": binding.PATH_COOPERATIVE, "staged": binding.PATH_STAGED}[args.path]
    staged = args.path == "staged" or (args.path == "auto" and w.M <= 8)
    kernel_name = ("distance_kernel + update_kernel (one round)" if args.path == "two_kernel" else
                   "round_kernel_staged (distance pass + grid barrier + update pass, one launch)" if staged else
                   "round_kernel (distance pass + grid barrier + update pass, one launch)")

    # CPU baseline first (rank 0, N = 1 only): before any GPU work, so the OpenMP team is
    # created in a process that has not touched CUDA yet.
    x_host = inputs.replicas(w, seed)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, cores, d_s, dt = time_oracle(w, x_host, budget_s=12.0)
        val1, _, d_1, dt1 = time_oracle(w, x_host, budget_s=6.0, threads=1)
        cpu = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"one oracle round on the first {d_s} of {w.d} columns ({dt:.1f} s), scaled by columns",
               "single_thread_value": val1}

    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    x_pinned = torch.from_numpy(x_host).pin_memory()
    x = binding.alloc_rows(w.M, w.d)
    x.copy_(x_pinned, non_blocking=True)
    norms = torch.zeros(w.M, device="cuda")
    ws = binding.alloc_workspace(w.M, w.d)
    B = w.M * w.d * 4
    fused = w.tau > 0          # local-step workload: every step = last local step fused with the round
    model_units = 7.0 if fused else 3.0      # x M d 4 bytes per step (two-pass fused round: 7, plain round: 3)
    if fused:
        v = binding.alloc_rows(w.M, w.d, fill=0.0)
        g = binding.alloc_rows(w.M, w.d)
        g.copy_(torch.from_numpy(inputs.gradients(w, 0, seed)).pin_memory(), non_blocking=True)
        staged = False
        kernel_name = ("distance_kernel<fused> + update_kernel (one step)" if args.path == "two_kernel" else
                       "round_kernel<fused> (local step + distance pass, grid barrier, update pass, one launch)")

    def step():
        if fused:
            binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay, w.alpha, w.lam,
                                                  norms_out=norms, ws=ws, d=w.d, path=path)
        else:
            binding.dppf_consensus(x, w.alpha, w.lam, norms_out=norms, ws=ws, d=w.d, path=path)

    def fence():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    fence()
    K = args.steps
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    with ClockSampler(physical_gpu_index(local)) as clocks:
        fence()
        ev[0].record()
        for i in range(K):
            step()
            ev[i + 1].record()
        fence()
    total_ms = ev[0].elapsed_time(ev[K])
    per_launch_ms = sum(ev[i].elapsed_time(ev[i + 1]) for i in range(K)) / K
    if binding.dppf_device_status(ws) != binding.OK:
        raise SystemExit("device status word reports an error")
    total_ms = max_over_ranks(total_ms, world, "cuda")
    launches_per_step = binding.launch_count(w.M, w.d, path, fused)

    # optional: the same K steps captured once into a CUDA graph and replayed (launch overhead off the host)
    graph_replay = None
    if args.graph:
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
    if not args.no_e2e and not fused:
        norms_host = torch.zeros(w.M).pin_memory()
        binding.dppf_consensus_host(x_pinned, w.alpha, w.lam, norms_host, x, ws, d=w.d)
        fence()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            binding.dppf_consensus_host(x_pinned, w.alpha, w.lam, norms_host, x, ws, d=w.d)
        e1.record()
        fence()
        e2e_ms = e0.elapsed_time(e1)
        e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
        e2e = {"value": whole_job_rate(args.e2e_steps, world, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": B, "d2h_bytes_per_step": B + 4 * w.M, "steps": args.e2e_steps}

    if rank == 0:
        peak, peak_src = measured_peaks()
        achieved = model_units * B / (per_launch_ms * 1e-3) / 1e9
        value = whole_job_rate(K, world, total_ms)
        model_gbs = model_units * B * K / (total_ms * 1e-3) / 1e9
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                "warmup": max(3, args.warmup), "ms_per_step": total_ms / K, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config_of(w, {"parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                                        "schedule": args.path}),
                "model_gbs_per_gpu": model_gbs, "frac_of_nominal_8tbs": model_gbs / NOMINAL_HBM_GBS,
                "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "traffic": measured_traffic(w, staged),
                             "kernel": kernel_name,
                             "algorithmic_bytes_per_launch": int(model_units) * B, "peak_source": f"of {peak_src}"},
                "clocks": clocks.summary(), "gpu_launches": K * launches_per_step,
                "norms_last_round": [float(v) for v in norms.cpu().tolist()]}
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
