"""CPU oracle for the DPPF consensus round -- TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper around ``dppf_oracle.c`` (plain C, fp64).  Only the test
suite, the smoke check and the benchmark's CPU-baseline legs may import this
package; the CUDA library and its Python binding never do, and this package
imports nothing from them.

Every function follows one passage of the paper:

* ``consensus``            -- the single-line pull-push update (Sec. 5), with
  ``x_A`` as defined on the last line of Algorithm 1 and every worker updated
  from the same pre-round average (first display in the proof of Theorem 1).
* ``consensus_two_step``   -- the pull line then the push line of Algorithm 1.
* ``local_steps_then_consensus`` -- tau local momentum-SGD steps (reading of
  the optimiser stated in ``dppf_oracle.c``) followed by the round.
* ``consensus_blocked``    -- the same round with the sum over coordinates
  grouped into per-thread column blocks (OpenMP), for timing and large cases.
* ``worker_update``        -- the single-line update (Sec. 5) of ONE worker given the
  average, as each worker applies it in Algorithm 1 after the collective (numpy, fp64).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dppf_oracle.c")
_LIB = os.path.join(_HERE, "libdppf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``dppf_oracle.c`` with gcc (no fused multiply-add contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        i64, i32, f32 = ctypes.c_int64, ctypes.c_int, ctypes.c_float
        common = [f32p, i32, i64, i64, f32, f32, f32p, i64, f64p]
        lib.dppf_oracle_consensus.argtypes = common
        lib.dppf_oracle_consensus_two_step.argtypes = common
        lib.dppf_oracle_consensus_f64.argtypes = [f64p, i32, i64, i64, f32, f32, f32p, i64, f64p]
        lib.dppf_oracle_consensus_blocked.argtypes = common + [i32, ctypes.POINTER(i32)]
        lib.dppf_oracle_local_step_f64.argtypes = [f64p, f64p, f32p, i32, i64, i64, i64, f32, f32, f32]
        lib.dppf_oracle_consensus_general.argtypes = [f32p, i32, i64, i64, f32, f32, f32p, i32, i32,
                                                      f32p, i64, f64p, f64p]
        lib.dppf_oracle_consensus_general.restype = i32
        lib.dppf_oracle_adamw_step_f64.argtypes = [f64p, f64p, f64p, f32p, i32, i64, i64, i64,
                                                   f32, f32, f32, f32, f32, i32]
        lib.dppf_oracle_adamw_step_f64.restype = i32
        for fn in (lib.dppf_oracle_consensus, lib.dppf_oracle_consensus_two_step,
                   lib.dppf_oracle_consensus_f64, lib.dppf_oracle_consensus_blocked,
                   lib.dppf_oracle_local_step_f64):
            fn.restype = i32
        _lib = lib
    return _lib


def _f32p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _f64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _check_2d(x, dtype):
    if x.dtype != dtype or x.ndim != 2 or x.strides[1] != x.itemsize or x.strides[0] % x.itemsize:
        raise ValueError(f"expected a 2-D {dtype} array with unit column stride")
    return x.shape[0], x.strides[0] // x.itemsize


def _run(fn, x, d, alpha, lam, extra=()):
    M, ld = _check_2d(x, np.float32)
    d = x.shape[1] if d is None else int(d)
    out = np.array(x, copy=True, order="C")          # pad columns carried over untouched
    r = np.zeros(M, dtype=np.float64)
    rc = fn(_f32p(x), M, d, ld, np.float32(alpha), np.float32(lam),
            _f32p(out), out.strides[0] // 4, _f64p(r), *extra)
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, r


def consensus(x, alpha, lam, d=None):
    """One pull-push round on fp32 replicas ``x[M, >=d]``; returns (x_plus fp32, r fp64)."""
    return _run(_load().dppf_oracle_consensus, x, d, alpha, lam)


def consensus_two_step(x, alpha, lam, d=None):
    """Algorithm 1's pull line followed by its push line."""
    return _run(_load().dppf_oracle_consensus_two_step, x, d, alpha, lam)


def consensus_blocked(x, alpha, lam, d=None, threads=0):
    """Column-block parallel round; returns (x_plus, r, threads_used)."""
    used = ctypes.c_int(0)
    out, r = _run(_load().dppf_oracle_consensus_blocked, x, d, alpha, lam,
                  extra=(int(threads), ctypes.byref(used)))
    return out, r, used.value


def consensus_general(x, alpha, lam, weights=None, push_from="average", two_term=False, d=None):
    """Algorithm 1 with a general consensus variable x_C = sum w_i x_i / sum w_i, the push
    taken from x_A ("average") or from x_C ("consensus"), and optionally both terms of the
    regulariser's gradient.  Returns (x_plus fp32, r fp64 = ||x_m - x_A||, n fp64 = ||y_m - P||)."""
    M, ld = _check_2d(x, np.float32)
    d = x.shape[1] if d is None else int(d)
    out = np.array(x, copy=True, order="C")
    r, n = np.zeros(M), np.zeros(M)
    wp = None
    if weights is not None:
        w32 = np.ascontiguousarray(np.asarray(weights, dtype=np.float32))
        if w32.shape != (M,):
            raise ValueError("weights must have one entry per worker")
        wp = _f32p(w32)
    rc = _load().dppf_oracle_consensus_general(
        _f32p(x), M, d, ld, np.float32(alpha), np.float32(lam), wp,
        {"average": 0, "consensus": 1}[push_from], int(bool(two_term)),
        _f32p(out), out.strides[0] // 4, _f64p(r), _f64p(n))
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, r, n


def local_steps_f64(x, v, grads, lr, momentum, weight_decay, d=None):
    """Apply ``len(grads)`` local steps in fp64.  ``x``, ``v`` are widened copies
    of the fp32 state (or already fp64); ``grads`` is an iterable of fp32
    ``[M, >=d]`` arrays, one per step.  Returns the fp64 state (x, v)."""
    x64 = np.array(x, dtype=np.float64, order="C")
    v64 = np.array(v, dtype=np.float64, order="C")
    M, ld = _check_2d(x64, np.float64)
    d = x64.shape[1] if d is None else int(d)
    lib = _load()
    for g in grads:
        Mg, ldg = _check_2d(g, np.float32)
        if Mg != M or g.shape[1] < d:
            raise ValueError("gradient shape mismatch")
        rc = lib.dppf_oracle_local_step_f64(_f64p(x64), _f64p(v64), _f32p(g), M, d, ld, ldg,
                                            np.float32(lr), np.float32(momentum),
                                            np.float32(weight_decay))
        if rc != 0:
            raise RuntimeError(f"oracle returned {rc}")
    return x64, v64


def adamw_steps_f64(x, m1, m2, grads, lr, beta1, beta2, eps, weight_decay, first_step=1, d=None):
    """Apply ``len(grads)`` AdamW steps (step numbers first_step, first_step+1, ...) in fp64.
    Returns the fp64 state (x, exp_avg, exp_avg_sq)."""
    x64 = np.array(x, dtype=np.float64, order="C")
    a64 = np.array(m1, dtype=np.float64, order="C")
    b64 = np.array(m2, dtype=np.float64, order="C")
    M, ld = _check_2d(x64, np.float64)
    d = x64.shape[1] if d is None else int(d)
    lib = _load()
    for k, g in enumerate(grads):
        Mg, ldg = _check_2d(g, np.float32)
        if Mg != M or g.shape[1] < d:
            raise ValueError("gradient shape mismatch")
        rc = lib.dppf_oracle_adamw_step_f64(_f64p(x64), _f64p(a64), _f64p(b64), _f32p(g), M, d, ld, ldg,
                                            np.float32(lr), np.float32(beta1), np.float32(beta2),
                                            np.float32(eps), np.float32(weight_decay), int(first_step) + k)
        if rc != 0:
            raise RuntimeError(f"oracle returned {rc}")
    return x64, a64, b64


def consensus_f64(x64, alpha, lam, d=None):
    """One round on an fp64 state; returns (x_plus fp32 [M, d], r fp64)."""
    M, ld = _check_2d(x64, np.float64)
    d = x64.shape[1] if d is None else int(d)
    out = np.zeros((M, d), dtype=np.float32)
    r = np.zeros(M, dtype=np.float64)
    rc = _load().dppf_oracle_consensus_f64(_f64p(x64), M, d, ld, np.float32(alpha),
                                           np.float32(lam), _f32p(out), d, _f64p(r))
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, r


def local_steps_then_consensus(x, v, grads, lr, momentum, weight_decay, alpha, lam, d=None):
    """tau local steps kept in fp64, then the round.  Returns
    (x_plus fp32 [M, d], v fp64 [M, ld], r fp64)."""
    x64, v64 = local_steps_f64(x, v, grads, lr, momentum, weight_decay, d)
    out, r = consensus_f64(x64, alpha, lam, d)
    return out, v64, r


def worker_update(x, reduced, scale, alpha, lam):
    """One worker's pull-push update given the all-reduced parameters (Algorithm 1 after
    "obtain x_C" with x_C = x_A; Sec. 5 single-line update): x_A = scale * reduced,
    r = ||x - x_A||, x_plus = x + (x_A - x)(alpha - lam / r); r == 0 leaves x as it is.
    ``x`` and ``reduced`` are fp32 vectors, the scalars are rounded to fp32 first (they cross
    the C ABI as floats) and everything else is fp64.  Returns (x_plus fp32, r fp64)."""
    x32 = np.asarray(x, dtype=np.float32)
    a_vec = np.float64(np.float32(scale)) * np.asarray(reduced, dtype=np.float32).astype(np.float64)
    x64 = x32.astype(np.float64)
    gap = a_vec - x64
    r = float(np.sqrt(np.sum(gap * gap)))
    if not r > 0.0:
        return x32.copy(), 0.0
    c = np.float64(np.float32(alpha)) - np.float64(np.float32(lam)) / r
    return (x64 + gap * c).astype(np.float32), r
