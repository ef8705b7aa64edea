"""The give-up path of the bounded waits, driven on a healthy GPU.

The staged kernels wait for their asynchronous row copies with a bounded number of polls.
dppf_debug_set_poll_limits(0, ...) makes every such wait of the distance pass give up at once
(or, with (default, 0), every wait of an update pass) while the copies themselves still
complete: a block that gives up waits for its copies in flight with the full budget before it
leaves.  Nothing faults or hangs; the call returns promptly and reports DPPF_ERR_TIMEOUT
through the status word."""
import time

import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev

pytestmark = pytest.mark.gpu


def replicas(M, d, seed):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * 0.02
    return padded((x0[None, :] + rng.standard_normal((M, d)) * 1e-3).astype(np.float32))


def calls(binding):
    """name -> (M, function(x, ws, d) issuing one call of a kernel that stages rows through shared memory)"""
    return {
        "round_staged_M4": (4, lambda x, ws, d: binding.dppf_consensus(x, 0.1, 0.01, ws=ws, d=d, path=3)),
        "round_staged_M16": (16, lambda x, ws, d: binding.dppf_consensus(x, 0.1, 0.01, ws=ws, d=d, path=3)),
        "rounds_M4": (4, lambda x, ws, d: binding.dppf_consensus_rounds(x, 0.1, 0.01, 3, ws=ws, d=d, path=3)),
        "rounds_M8": (8, lambda x, ws, d: binding.dppf_consensus_rounds(x, 0.1, 0.01, 2, ws=ws, d=d, path=3)),
        "general_M4": (4, lambda x, ws, d: binding.dppf_consensus_general(x, 0.1, 0.01, [1, 2, 3, 4], 1, True, ws=ws,
                                                                          d=d, path=3)),
    }


NAMES = ["round_staged_M4", "round_staged_M16", "rounds_M4", "rounds_M8", "general_M4"]


@pytest.mark.parametrize("name", NAMES)
def test_give_up_in_the_distance_pass_leaves_x_untouched(oracle, name):
    import torch
    _, binding = require_gpu()
    M, call = calls(binding)[name]
    d = 1_000_003
    x_np = replicas(M, d, seed=len(name))
    x = to_dev(x_np)
    ws = binding.alloc_workspace(M, d)
    try:
        binding.debug_set_poll_limits(0, -1)
        t0 = time.perf_counter()
        call(x, ws, d)
        status = binding.dppf_device_status(ws)          # synchronises the stream
        elapsed = time.perf_counter() - t0
    finally:
        binding.debug_set_poll_limits(-1, -1)
    assert status == binding.ERR_TIMEOUT
    assert elapsed < 5.0
    assert same_bits(x.cpu().numpy()[:, :d], x_np[:, :d])
    assert_pad_untouched(x.cpu().numpy(), d)
    # the next ordinary call on the same workspace is correct and clears the status
    norms = torch.zeros(M, device="cuda")
    binding.dppf_consensus(x, 0.1, 0.01, norms_out=norms, ws=ws, d=d, path=3)
    assert binding.dppf_device_status(ws) == binding.OK
    ref, r_ref = oracle.consensus(x_np, 0.1, 0.01, d=d)
    got = x.cpu().numpy()
    assert_parity(got, norms.cpu().numpy(), ref, r_ref, d)
    assert_pad_untouched(got, d)


@pytest.mark.parametrize("name", NAMES)
def test_give_up_in_an_update_pass_is_reported(oracle, name):
    import torch
    _, binding = require_gpu()
    M, call = calls(binding)[name]
    d = 6_000_005            # every block has more chunks than ring stages, so update passes do wait
    x_np = replicas(M, d, seed=100 + len(name))
    x = to_dev(x_np)
    ws = binding.alloc_workspace(M, d)
    try:
        binding.debug_set_poll_limits(-1, 0)
        call(x, ws, d)
        status = binding.dppf_device_status(ws)
    finally:
        binding.debug_set_poll_limits(-1, -1)
    assert status == binding.ERR_TIMEOUT
    assert_pad_untouched(x.cpu().numpy(), d)             # partly updated, but never outside the rows
    # same buffers, ordinary call from a fresh copy of the input
    x.copy_(torch.from_numpy(x_np))
    norms = torch.zeros(M, device="cuda")
    binding.dppf_consensus(x, 0.1, 0.01, norms_out=norms, ws=ws, d=d)
    assert binding.dppf_device_status(ws) == binding.OK
    ref, r_ref = oracle.consensus(x_np, 0.1, 0.01, d=d)
    assert_parity(x.cpu().numpy(), norms.cpu().numpy(), ref, r_ref, d)


@pytest.mark.parametrize("limits", [(0, -1), (-1, 0)])
def test_give_up_in_the_fused_local_step_round_is_reported(oracle, limits):
    """The staged kernel that fuses the last SGD-momentum step with the round: its first pass
    already rewrites x and v, so a give-up leaves them partly stepped; what is promised is the
    status word, rows that stay inside their bounds, and a working library afterwards."""
    import torch
    from paper_2507_20424_b200 import inputs
    _, binding = require_gpu()
    M, d = 4, 6_000_005
    w = inputs.WORKLOADS["C3"].scaled(d)
    x_np, v_np, g_np = inputs.replicas(w), inputs.zeros_like_rows(w), inputs.gradients(w, 0)
    x_np[:, :d] += inputs.gradients(w, 3)[:, :d]
    x, v, g = to_dev(x_np), to_dev(v_np), to_dev(g_np)
    ws = binding.alloc_workspace(M, d)
    try:
        binding.debug_set_poll_limits(*limits)
        binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay, w.alpha, w.lam, ws=ws, d=d,
                                              path=3)
        status = binding.dppf_device_status(ws)
    finally:
        binding.debug_set_poll_limits(-1, -1)
    assert status == binding.ERR_TIMEOUT
    assert_pad_untouched(x.cpu().numpy(), d), assert_pad_untouched(v.cpu().numpy(), d)
    x.copy_(torch.from_numpy(x_np)), v.copy_(torch.from_numpy(v_np))
    norms = torch.zeros(M, device="cuda")
    binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay, w.alpha, w.lam, norms_out=norms,
                                          ws=ws, d=d, path=3)
    assert binding.dppf_device_status(ws) == binding.OK
    ref, _, r_ref = oracle.local_steps_then_consensus(x_np[:, :d], v_np[:, :d], [g_np[:, :d]], w.lr, w.momentum,
                                                      w.weight_decay, w.alpha, w.lam)
    assert_parity(x.cpu().numpy(), norms.cpu().numpy(), ref, r_ref, d)


def test_default_budget_is_restored():
    _, binding = require_gpu()
    d = 300_001
    x_np = replicas(4, d, seed=5)
    x = to_dev(x_np)
    ws = binding.alloc_workspace(4, d)
    binding.debug_set_poll_limits(0, 0)
    binding.debug_set_poll_limits(-1, -1)
    binding.dppf_consensus_rounds(x, 0.1, 0.01, 2, ws=ws, d=d)
    assert binding.dppf_device_status(ws) == binding.OK
    assert not same_bits(x.cpu().numpy()[:, :d], x_np[:, :d])
