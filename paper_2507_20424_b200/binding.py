"""ctypes binding of ``libdppf.so``: argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory) and
passes raw pointers, sizes and the current CUDA stream to the C entry point of
the same name (``include/dppf.h``).  There is no CPU fallback: if the library
is missing or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

PATH_AUTO, PATH_TWO_KERNEL, PATH_COOPERATIVE, PATH_STAGED = 0, 1, 2, 3
OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)

EXPORTS = ("dppf_workspace_bytes", "dppf_consensus", "dppf_consensus_ex", "dppf_local_step",
           "dppf_local_step_and_consensus", "dppf_local_step_and_consensus_ex",
           "dppf_consensus_host", "dppf_device_status", "dppf_device_schedule", "dppf_status_string", "dppf_launch_count",
           "dppf_consensus_static", "dppf_static_device_status", "dppf_consensus_general", "dppf_consensus_general_ex",
           "dppf_distance_partials", "dppf_update_from_sums", "dppf_worker_update", "dppf_adamw_step_and_consensus_ex",
           "dppf_consensus_rounds", "dppf_consensus_rounds_ex", "dppf_debug_set_poll_limits",
           "dppf_adamw_step", "dppf_adamw_step_and_consensus",
           "dppf_lambda_schedule", "dppf_lr_cosine", "dppf_qsr_period", "dppf_round_metrics")

_lib = None


class DppfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def library_path() -> str:
    return _build.LIB_PATH


def load(rebuild_if_stale: bool = False) -> ctypes.CDLL:
    """Load the shared library (building it first only when asked to)."""
    global _lib
    if _lib is not None:
        return _lib
    if rebuild_if_stale:
        _build.build()
    if not os.path.exists(_build.LIB_PATH):
        raise RuntimeError(f"{_build.LIB_PATH} not found: build it with "
                           "`python -m paper_2507_20424_b200.build` (no CPU fallback exists)")
    lib = ctypes.CDLL(_build.LIB_PATH)
    vp, f32, i32, i64, sz = ctypes.c_void_p, ctypes.c_float, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.dppf_workspace_bytes.argtypes = [i32, i64]
    lib.dppf_workspace_bytes.restype = sz
    lib.dppf_consensus.argtypes = [vp, i32, i64, i64, f32, f32, vp, vp, sz, vp]
    lib.dppf_consensus_ex.argtypes = [vp, i32, i64, i64, f32, f32, vp, vp, sz, i32, vp]
    lib.dppf_local_step.argtypes = [vp, vp, vp, i32, i64, i64, f32, f32, f32, vp]
    lib.dppf_local_step_and_consensus.argtypes = [vp, vp, vp, i32, i64, i64, f32, f32, f32, f32, f32, vp, vp, sz, vp]
    lib.dppf_local_step_and_consensus_ex.argtypes = [vp, vp, vp, i32, i64, i64, f32, f32, f32, f32, f32, vp, vp, sz, i32, vp]
    lib.dppf_consensus_host.argtypes = [vp, i32, i64, i64, f32, f32, vp, vp, vp, sz, vp]
    lib.dppf_device_status.argtypes = [vp, vp]
    lib.dppf_device_schedule.argtypes = [vp, vp]
    lib.dppf_device_schedule.restype = i32
    lib.dppf_lambda_schedule.argtypes = [i32, f32, i64, i64]
    lib.dppf_lambda_schedule.restype = f32
    lib.dppf_lr_cosine.argtypes = [f32, i64, i64]
    lib.dppf_lr_cosine.restype = f32
    lib.dppf_qsr_period.argtypes = [i64, f32, f32]
    lib.dppf_qsr_period.restype = i64
    lib.dppf_round_metrics.argtypes = [ctypes.POINTER(f32), i32, f32, f32, ctypes.POINTER(f32),
                                       ctypes.POINTER(f32), ctypes.POINTER(f32)]
    lib.dppf_round_metrics.restype = i32
    lib.dppf_adamw_step.argtypes = [vp, vp, vp, vp, i32, i64, i64, f32, f32, f32, f32, f32, i32, vp]
    lib.dppf_adamw_step.restype = i32
    lib.dppf_adamw_step_and_consensus.argtypes = [vp, vp, vp, vp, i32, i64, i64, f32, f32, f32, f32, f32, i32,
                                                  f32, f32, vp, vp, sz, vp]
    lib.dppf_adamw_step_and_consensus.restype = i32
    lib.dppf_consensus_general.argtypes = [vp, i32, i64, i64, f32, f32, ctypes.POINTER(f32), i32, i32, vp, vp,
                                           vp, sz, vp]
    lib.dppf_consensus_general.restype = i32
    lib.dppf_consensus_rounds.argtypes = [vp, i32, i64, i64, f32, f32, ctypes.POINTER(f32), i32, vp, vp, sz, vp]
    lib.dppf_consensus_rounds.restype = i32
    lib.dppf_consensus_rounds_ex.argtypes = [vp, i32, i64, i64, f32, f32, ctypes.POINTER(f32), i32, vp, vp, sz,
                                             i32, vp]
    lib.dppf_consensus_rounds_ex.restype = i32
    lib.dppf_distance_partials.argtypes = [vp, i32, i64, i64, vp, vp, sz, vp]
    lib.dppf_distance_partials.restype = i32
    lib.dppf_update_from_sums.argtypes = [vp, i32, i64, i64, f32, f32, vp, vp, vp]
    lib.dppf_update_from_sums.restype = i32
    lib.dppf_worker_update.argtypes = [vp, vp, f32, i64, f32, f32, vp, vp, sz, vp]
    lib.dppf_worker_update.restype = i32
    lib.dppf_static_device_status.argtypes = [vp]
    lib.dppf_static_device_status.restype = i32
    lib.dppf_consensus_general_ex.argtypes = [vp, i32, i64, i64, f32, f32, ctypes.POINTER(f32), i32, i32, vp, vp,
                                              vp, sz, i32, vp]
    lib.dppf_consensus_general_ex.restype = i32
    lib.dppf_adamw_step_and_consensus_ex.argtypes = [vp, vp, vp, vp, i32, i64, i64, f32, f32, f32, f32, f32, i32,
                                                     f32, f32, vp, vp, sz, i32, vp]
    lib.dppf_adamw_step_and_consensus_ex.restype = i32
    lib.dppf_debug_set_poll_limits.argtypes = [i32, i32]
    lib.dppf_debug_set_poll_limits.restype = i32
    lib.dppf_consensus_static.argtypes = [vp, i32, i64, i64, f32, f32, vp, vp]
    lib.dppf_consensus_static.restype = i32
    lib.dppf_status_string.argtypes = [i32]
    lib.dppf_status_string.restype = ctypes.c_char_p
    lib.dppf_launch_count.argtypes = [i32, i64, i32, i32]
    for name in ("dppf_consensus", "dppf_consensus_ex", "dppf_local_step", "dppf_local_step_and_consensus",
                 "dppf_local_step_and_consensus_ex", "dppf_consensus_host", "dppf_device_status", "dppf_device_schedule",
                 "dppf_launch_count"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().dppf_status_string(int(status)).decode()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise DppfError(rc, where)


def _dims(x: torch.Tensor, d):
    if x.dim() != 2 or x.dtype != torch.float32 or not x.is_cuda or x.stride(1) != 1:
        raise ValueError("expected a 2-D fp32 CUDA tensor with unit column stride")
    M, ld = x.shape[0], x.stride(0)
    return M, (x.shape[1] if d is None else int(d)), ld


def workspace_bytes(M: int, d: int) -> int:
    return int(load().dppf_workspace_bytes(int(M), int(d)))


def alloc_workspace(M: int, d: int, device="cuda") -> torch.Tensor:
    n = workspace_bytes(M, d)
    if n == 0:
        raise ValueError("invalid M or d")
    return torch.empty(n, dtype=torch.uint8, device=device)


def alloc_rows(M: int, d: int, device="cuda", fill=None) -> torch.Tensor:
    """[M, ld] fp32 device buffer with 128-byte rows (ld = d rounded up to 32)."""
    ld = (int(d) + 31) // 32 * 32
    t = torch.empty((M, ld), dtype=torch.float32, device=device)
    if fill is not None:
        t.fill_(fill)
    return t


def _ptr(t):
    return None if t is None else t.data_ptr()


def dppf_consensus(x, alpha, lam, norms_out=None, ws=None, d=None, path=PATH_AUTO):
    """One pull-push round in place on ``x[M, ld]``; returns the workspace used."""
    M, d, ld = _dims(x, d)
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    rc = load().dppf_consensus_ex(x.data_ptr(), M, d, ld, alpha, lam, _ptr(norms_out),
                                  ws.data_ptr(), ws.numel(), int(path), _stream())
    _check(rc, "dppf_consensus")
    return ws


def dppf_consensus_rounds(x, alpha, lam, n_rounds, lambdas=None, norms_out=None, ws=None, d=None, path=PATH_AUTO):
    """``n_rounds`` rounds in place on ``x[M, ld]`` in one pass sequence; ``lambdas`` (host
    sequence of n_rounds floats) overrides ``lam`` per round; ``norms_out`` is [n_rounds, M]."""
    M, d, ld = _dims(x, d)
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    lp = None
    if lambdas is not None:
        if len(lambdas) != n_rounds:
            raise ValueError("lambdas must have one entry per round")
        lp = (ctypes.c_float * n_rounds)(*[float(v) for v in lambdas])
    if norms_out is not None and norms_out.numel() < n_rounds * M:
        raise ValueError("norms_out must hold n_rounds x M floats")
    rc = load().dppf_consensus_rounds_ex(x.data_ptr(), M, d, ld, alpha, lam, lp, int(n_rounds), _ptr(norms_out),
                                         ws.data_ptr(), ws.numel(), int(path), _stream())
    _check(rc, "dppf_consensus_rounds")
    return ws


def dppf_distance_partials(x, sums_out, ws=None, d=None):
    """Sums of squared distances to the column average over this column shard -> ``sums_out``
    (fp64 CUDA tensor of M entries).  Returns the workspace used."""
    M, d, ld = _dims(x, d)
    if sums_out.dtype != torch.float64 or not sums_out.is_cuda or sums_out.numel() < M:
        raise ValueError("sums_out must be an fp64 CUDA tensor with M entries")
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    _check(load().dppf_distance_partials(x.data_ptr(), M, d, ld, sums_out.data_ptr(), ws.data_ptr(), ws.numel(),
                                         _stream()), "dppf_distance_partials")
    return ws


def dppf_update_from_sums(x, alpha, lam, sums, norms_out=None, d=None):
    """Update pass on this column shard from the sums of squares totalled over all shards."""
    M, d, ld = _dims(x, d)
    if sums.dtype != torch.float64 or not sums.is_cuda or sums.numel() < M:
        raise ValueError("sums must be an fp64 CUDA tensor with M entries")
    _check(load().dppf_update_from_sums(x.data_ptr(), M, d, ld, alpha, lam, sums.data_ptr(), _ptr(norms_out),
                                        _stream()), "dppf_update_from_sums")


def dppf_worker_update(x, x_reduced, scale, alpha, lam, norm_out=None, ws=None):
    """This worker's pull-push update from the all-reduced parameters (one replica per GPU):
    ``x`` and ``x_reduced`` are 1-D fp32 CUDA tensors of the same length; x_A = scale * x_reduced."""
    for t in (x, x_reduced):
        if t.dim() != 1 or t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("expected contiguous 1-D fp32 CUDA tensors")
    if x.numel() != x_reduced.numel():
        raise ValueError("x and x_reduced must have the same length")
    d = x.numel()
    ws = alloc_workspace(1, d, x.device) if ws is None else ws
    _check(load().dppf_worker_update(x.data_ptr(), x_reduced.data_ptr(), scale, d, alpha, lam, _ptr(norm_out),
                                     ws.data_ptr(), ws.numel(), _stream()), "dppf_worker_update")
    return ws


def debug_set_poll_limits(first_pass_polls=-1, later_pass_polls=-1) -> None:
    """Testing hook: poll budget of the bounded waits of later calls (negative = default)."""
    load().dppf_debug_set_poll_limits(int(first_pass_polls), int(later_pass_polls))


PUSH_FROM_AVERAGE, PUSH_FROM_CONSENSUS = 0, 1


def dppf_consensus_general(x, alpha, lam, weights=None, push_from=PUSH_FROM_AVERAGE, two_term=False,
                           norms_out=None, push_norms_out=None, ws=None, d=None, path=PATH_AUTO):
    """General round in place on ``x[M, ld]``: consensus variable from ``weights`` (host
    sequence of M floats, None = plain average), push from x_A or x_C, optional second term."""
    M, d, ld = _dims(x, d)
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    wp = None
    if weights is not None:
        if len(weights) != M:
            raise ValueError("weights must have one entry per worker")
        wp = (ctypes.c_float * M)(*[float(v) for v in weights])
    rc = load().dppf_consensus_general_ex(x.data_ptr(), M, d, ld, alpha, lam, wp, int(push_from),
                                          int(bool(two_term)), _ptr(norms_out), _ptr(push_norms_out),
                                          ws.data_ptr(), ws.numel(), int(path), _stream())
    _check(rc, "dppf_consensus_general")
    return ws


def dppf_consensus_static(x, alpha, lam, norms_out=None, d=None):
    """One round in place on ``x[M, ld]`` using the library's built-in scratch: no
    workspace argument and no allocation anywhere in the call (M <= 16).  Calls that
    may overlap on the GPU must be ordered by the caller; they share the scratch."""
    M, d, ld = _dims(x, d)
    rc = load().dppf_consensus_static(x.data_ptr(), M, d, ld, alpha, lam, _ptr(norms_out), _stream())
    _check(rc, "dppf_consensus_static")


def dppf_local_step(x, v, g, lr, momentum, weight_decay, d=None):
    M, d, ld = _dims(x, d)
    for t in (v, g):
        if _dims(t, d) != (M, d, ld):
            raise ValueError("x, v and g must share shape and row stride")
    _check(load().dppf_local_step(x.data_ptr(), v.data_ptr(), g.data_ptr(), M, d, ld,
                                  lr, momentum, weight_decay, _stream()), "dppf_local_step")


def dppf_local_step_and_consensus(x, v, g, lr, momentum, weight_decay, alpha, lam,
                                  norms_out=None, ws=None, d=None, path=PATH_AUTO):
    M, d, ld = _dims(x, d)
    for t in (v, g):
        if _dims(t, d) != (M, d, ld):
            raise ValueError("x, v and g must share shape and row stride")
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    rc = load().dppf_local_step_and_consensus_ex(
        x.data_ptr(), v.data_ptr(), g.data_ptr(), M, d, ld, lr, momentum, weight_decay,
        alpha, lam, _ptr(norms_out), ws.data_ptr(), ws.numel(), int(path), _stream())
    _check(rc, "dppf_local_step_and_consensus")
    return ws


def _same_shape(x, others, d):
    M, d, ld = _dims(x, d)
    for t in others:
        if _dims(t, d) != (M, d, ld):
            raise ValueError("all buffers must share shape and row stride")
    return M, d, ld


def dppf_adamw_step(x, exp_avg, exp_avg_sq, g, lr, beta1, beta2, eps, weight_decay, step, d=None):
    M, d, ld = _same_shape(x, (exp_avg, exp_avg_sq, g), d)
    _check(load().dppf_adamw_step(x.data_ptr(), exp_avg.data_ptr(), exp_avg_sq.data_ptr(), g.data_ptr(), M, d, ld,
                                  lr, beta1, beta2, eps, weight_decay, int(step), _stream()), "dppf_adamw_step")


def dppf_adamw_step_and_consensus(x, exp_avg, exp_avg_sq, g, lr, beta1, beta2, eps, weight_decay, step,
                                  alpha, lam, norms_out=None, ws=None, d=None, path=PATH_AUTO):
    M, d, ld = _same_shape(x, (exp_avg, exp_avg_sq, g), d)
    ws = alloc_workspace(M, d, x.device) if ws is None else ws
    rc = load().dppf_adamw_step_and_consensus_ex(
        x.data_ptr(), exp_avg.data_ptr(), exp_avg_sq.data_ptr(), g.data_ptr(), M, d, ld, lr, beta1, beta2, eps,
        weight_decay, int(step), alpha, lam, _ptr(norms_out), ws.data_ptr(), ws.numel(), int(path), _stream())
    _check(rc, "dppf_adamw_step_and_consensus")
    return ws


def dppf_consensus_host(x_host, alpha, lam, norms_host, x_dev, ws, d=None):
    """Round on host-resident replicas (pinned CPU tensors), staged through ``x_dev``."""
    M, d, ld = _dims(x_dev, d)
    if x_host.dtype != torch.float32 or x_host.is_cuda or x_host.shape[0] != M or x_host.stride(0) != ld:
        raise ValueError("x_host must be a CPU fp32 tensor with the row stride of x_dev")
    rc = load().dppf_consensus_host(x_host.data_ptr(), M, d, ld, alpha, lam, _ptr(norms_host),
                                    x_dev.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    _check(rc, "dppf_consensus_host")


SCHEDULE_FIXED, SCHEDULE_DECREASING, SCHEDULE_INCREASING = 0, 1, 2


def dppf_lambda_schedule(kind, lam, t, T) -> float:
    return float(load().dppf_lambda_schedule(int(kind), lam, int(t), int(T)))


def dppf_lr_cosine(lr_max, t, T) -> float:
    return float(load().dppf_lr_cosine(lr_max, int(t), int(T)))


def dppf_qsr_period(tau_base, beta, lr_t) -> int:
    return int(load().dppf_qsr_period(int(tau_base), beta, lr_t))


def dppf_round_metrics(norms, alpha, lam):
    """(mean distance, [pull strength per worker], push strength) from host distances."""
    M = len(norms)
    arr = (ctypes.c_float * M)(*[float(v) for v in norms])
    pull = (ctypes.c_float * M)()
    mean, push = ctypes.c_float(), ctypes.c_float()
    _check(load().dppf_round_metrics(arr, M, alpha, lam, ctypes.byref(mean), pull, ctypes.byref(push)),
           "dppf_round_metrics")
    return mean.value, list(pull), push.value


def dppf_device_status(ws) -> int:
    return int(load().dppf_device_status(ws.data_ptr(), _stream()))


def dppf_device_schedule(ws) -> int:
    """PATH_* of the kernels that ran the last call on this workspace (synchronises the stream)."""
    return int(load().dppf_device_schedule(ws.data_ptr(), _stream()))


def launch_count(M: int, d: int, path=PATH_AUTO, fused=False) -> int:
    return int(load().dppf_launch_count(int(M), int(d), int(path), int(bool(fused))))


def adamw_launch_count(M: int, path=PATH_AUTO) -> int:
    """Kernel launches of one dppf_adamw_step_and_consensus call."""
    return int(load().dppf_launch_count(int(M), 1, int(path), 2))


def dppf_static_device_status() -> int:
    """Status word of the built-in scratch that dppf_consensus_static uses on the current device."""
    return int(load().dppf_static_device_status(_stream()))
