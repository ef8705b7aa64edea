"""dppf_consensus_static: the round for callers that cannot allocate device memory
(code running under a fixed memory budget, or handed pointers by a host that owns the
allocator).  It keeps its per-block partial sums in an array inside the library instead
of a caller workspace.  The file name sorts last on purpose: a run that stops at the first
failure has then already run every other test.

Checked here, through the C ABI: the result equals dppf_consensus's on the same input, on
two calls in a row (the second one finds the first one's leftovers in the shared array,
with a different worker count and grid), and a worker count above the limit is refused."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev

pytestmark = pytest.mark.gpu


def _replicas(M, d, seed):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * 0.02
    return padded((x0[None, :] + rng.standard_normal((M, d)) * 1e-3).astype(np.float32))


def _both(binding, x_np, d, alpha, lam):
    import torch
    M = x_np.shape[0]
    xa, xb = to_dev(x_np), to_dev(x_np)
    na, nb = torch.full((M,), -1.0, device="cuda"), torch.full((M,), -2.0, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus(xa, alpha, lam, norms_out=na, ws=ws, d=d)
    binding.dppf_consensus_static(xb, alpha, lam, norms_out=nb, d=d)
    torch.cuda.synchronize()
    return xa.cpu().numpy(), na.cpu().numpy(), xb.cpu().numpy(), nb.cpu().numpy()


def test_static_scratch_round_matches_workspace_round_twice_in_a_row(oracle):
    _, binding = require_gpu()
    # call 1: M = 8 on a long vector (full grid); call 2: M = 3 on a short ragged one (small
    # grid), so the second call runs over stale partial sums of the first
    for M, d, alpha, lam, seed in ((8, 3_000_017, 0.05, 0.02, 31), (3, 70_001, 0.1, 0.01, 32)):
        x_np = _replicas(M, d, seed)
        xa, na, xb, nb = _both(binding, x_np, d, alpha, lam)
        # tolerance of the parity tests; the two entry points in fact agree bit for bit
        ref = xa[:, :d].astype(np.float64)
        assert np.all(np.abs(xb[:, :d].astype(np.float64) - ref) <= 1e-6 * (1 + np.abs(ref)))
        assert np.all(np.abs(nb.astype(np.float64) - na) <= 1e-5 * na)
        assert same_bits(xa[:, :d], xb[:, :d]) and same_bits(na, nb)
        assert not same_bits(xb[:, :d], x_np[:, :d])          # the round did run
        assert_pad_untouched(xb, d)
        # and directly against the CPU oracle, at the tolerances of the parity tests
        ref, r_ref = oracle.consensus(x_np, alpha, lam, d=d)
        assert_parity(xb, nb, ref, r_ref, d)
        assert binding.dppf_static_device_status() == binding.OK


def test_static_scratch_round_repeats_and_works_without_norms():
    import torch
    _, binding = require_gpu()
    d = 400_003
    x_np = _replicas(4, d, 33)
    xa, xb = to_dev(x_np), to_dev(x_np)
    ws = binding.alloc_workspace(4, d)
    for _ in range(3):
        binding.dppf_consensus(xa, 0.1, 0.005, ws=ws, d=d)
        binding.dppf_consensus_static(xb, 0.1, 0.005, d=d)
    torch.cuda.synchronize()
    assert same_bits(xa.cpu().numpy()[:, :d], xb.cpu().numpy()[:, :d])


def test_static_scratch_calls_allocate_nothing():
    """Neither the driver's free-memory figure nor torch's allocator moves across warmed-up calls."""
    import torch
    _, binding = require_gpu()
    d = 1_000_003
    x = to_dev(_replicas(4, d, 35))
    norms = torch.zeros(4, device="cuda")
    binding.dppf_consensus_static(x, 0.1, 0.005, norms_out=norms, d=d)          # first call: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(5):
        binding.dppf_consensus_static(x, 0.1, 0.005, norms_out=norms, d=d)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert binding.dppf_static_device_status() == binding.OK


def test_static_scratch_status_word_reports_a_give_up():
    """The status word of the built-in scratch is readable without a workspace pointer: a wait
    that gives up in the staged kernel (poll budget 0, see test_gpu_timeouts.py) shows up there."""
    _, binding = require_gpu()
    d = 1_000_003
    x_np = _replicas(4, d, 36)
    x = to_dev(x_np)
    try:
        binding.debug_set_poll_limits(0, -1)
        binding.dppf_consensus_static(x, 0.1, 0.005, d=d)
        status = binding.dppf_static_device_status()
    finally:
        binding.debug_set_poll_limits(-1, -1)
    assert status == binding.ERR_TIMEOUT
    assert same_bits(x.cpu().numpy()[:, :d], x_np[:, :d])
    binding.dppf_consensus_static(x, 0.1, 0.005, d=d)
    assert binding.dppf_static_device_status() == binding.OK


def test_static_scratch_round_refuses_too_many_workers_and_bad_layout():
    import torch
    _, binding = require_gpu()
    x = to_dev(_replicas(17, 1000, 34))
    before = x.clone()
    with pytest.raises(binding.DppfError) as e:
        binding.dppf_consensus_static(x, 0.1, 0.01, d=1000)
    assert e.value.status == binding.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.equal(x.view(torch.int32), before.view(torch.int32))     # nothing was launched
    lib = binding.load()
    assert lib.dppf_consensus_static(None, 4, 64, 64, 0.1, 0.01, None, None) == binding.ERR_INVALID_ARG
    assert lib.dppf_consensus_static(0x10000000, 4, 60, 60, 0.1, 0.01, None, None) == binding.ERR_ALIGNMENT
