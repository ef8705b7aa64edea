"""Seeded synthetic inputs for the DPPF consensus round.

This module holds no arithmetic of the method itself: it only draws the
random replicas and gradients that both the CUDA path and the CPU checker are
fed with.  Real trained weights are not needed for this step -- a round acts
on flat parameter vectors, so Gaussian vectors with the parameter counts of
the paper's models (PyramidNet, ResNet-50/101, a ViT) stand in for them.

Random streams are Philox generators keyed by ``(seed, stream)``:

    stream 0            the shared initial point x0
    stream 1 + m        drift of worker m away from x0
    stream 99           per-worker drift scales (mixed-scale workload)
    stream 100+16*t+m   gradient of worker m at local step t

Arrays are ``[M, ld]`` fp32, ``ld = row_stride(d)`` (rows padded to 128 bytes);
pad columns hold ``PAD_VALUE`` (NaN) so that any read of them poisons a sum
and any write to them is visible.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np

DEFAULT_SEED = 20424
PAD_VALUE = np.float32("nan")


def row_stride(d: int) -> int:
    """Smallest multiple of 32 floats (128 bytes) that holds d columns."""
    return (int(d) + 31) // 32 * 32


@dataclass(frozen=True)
class Workload:
    name: str
    M: int
    d: int
    x0_std: float
    alpha: float
    lam: float
    drift_std: Optional[float] = None              # same scale for every worker
    drift_log10_range: Optional[Tuple[float, float]] = None   # per-worker log-uniform scale
    rounds: int = 1
    # local optimiser between rounds (None = consensus only)
    tau: int = 0
    lr: float = 0.0
    momentum: float = 0.0
    weight_decay: float = 0.0
    grad_std: float = 0.0
    model: str = ""

    @property
    def ld(self) -> int:
        return row_stride(self.d)

    def scaled(self, d: int) -> "Workload":
        """Same recipe on a shorter vector (for cases a CPU finishes quickly)."""
        return replace(self, d=int(d), name=f"{self.name}[d={int(d)}]")


WORKLOADS = {
    "C1": Workload("C1", M=4, d=1_048_576, x0_std=0.02, drift_std=1e-3,
                   alpha=0.1, lam=0.01, model="small"),
    "C2": Workload("C2", M=8, d=26_200_000, x0_std=0.05, drift_std=5e-3,
                   alpha=0.05, lam=0.02, model="PyramidNet-sized"),
    "C3": Workload("C3", M=4, d=25_557_032, x0_std=0.02, drift_std=None,
                   alpha=0.1, lam=0.01, tau=8, lr=0.1, momentum=0.9,
                   weight_decay=1e-4, grad_std=1e-2, model="ResNet-50-sized"),
    "C4": Workload("C4", M=4, d=86_567_656, x0_std=0.02, drift_std=1e-3,
                   alpha=0.1, lam=0.005, rounds=100, model="ViT-B/16-sized"),
    "C5": Workload("C5", M=16, d=44_549_160, x0_std=0.02,
                   drift_log10_range=(-5.0, -2.0), alpha=0.2, lam=0.05,
                   model="ResNet-101-sized"),
}


def _normal(seed: int, stream: int, n: int) -> np.ndarray:
    gen = np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))
    return gen.standard_normal(n, dtype=np.float32)


def drift_scales(w: Workload, seed: int = DEFAULT_SEED) -> np.ndarray:
    """Standard deviation of each worker's drift, fp64 [M]."""
    if w.drift_log10_range is not None:
        lo, hi = w.drift_log10_range
        u = np.random.Generator(np.random.Philox(key=[int(seed), 99])).random(w.M)
        return 10.0 ** (lo + (hi - lo) * u)
    if w.drift_std is None:
        return np.zeros(w.M)
    return np.full(w.M, float(w.drift_std))


def empty_rows(M: int, d: int) -> np.ndarray:
    """[M, ld] fp32 with every pad column set to PAD_VALUE."""
    ld = row_stride(d)
    a = np.empty((M, ld), dtype=np.float32)
    a[:, d:] = PAD_VALUE
    return a


def _fill_rows(out: np.ndarray, d: int, fn, threads: int) -> None:
    M = out.shape[0]
    if threads > 1 and M > 1:
        with ThreadPoolExecutor(max_workers=min(threads, M)) as ex:
            list(ex.map(lambda m: fn(m, out[m, :d]), range(M)))
    else:
        for m in range(M):
            fn(m, out[m, :d])


def replicas(w: Workload, seed: int = DEFAULT_SEED, identical: bool = False,
             threads: int = 8) -> np.ndarray:
    """Worker replicas ``x[M, ld]``: a shared x0 plus each worker's drift.
    ``identical=True`` gives M exact copies of x0 (the zero-distance round)."""
    x0 = _normal(seed, 0, w.d) * np.float32(w.x0_std)
    sig = drift_scales(w, seed)
    x = empty_rows(w.M, w.d)

    def fill(m, row):
        if identical or sig[m] == 0.0:
            row[:] = x0
        else:
            np.multiply(_normal(seed, 1 + m, w.d), np.float32(sig[m]), out=row)
            row += x0

    _fill_rows(x, w.d, fill, threads)
    return x


def zeros_like_rows(w: Workload) -> np.ndarray:
    """Momentum buffers ``v[M, ld]`` at their initial value 0."""
    v = empty_rows(w.M, w.d)
    v[:, :w.d] = 0.0
    return v


def gradients(w: Workload, step: int, seed: int = DEFAULT_SEED, threads: int = 8) -> np.ndarray:
    """Synthetic gradients ``g[M, ld]`` of all workers at local step ``step`` (0-based)."""
    g = empty_rows(w.M, w.d)

    def fill(m, row):
        np.multiply(_normal(seed, 100 + 16 * step + m, w.d), np.float32(w.grad_std), out=row)

    _fill_rows(g, w.d, fill, threads)
    return g
