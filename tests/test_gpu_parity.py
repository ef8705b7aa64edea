"""CUDA path vs the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev
from paper_2507_20424_b200 import inputs

pytestmark = pytest.mark.gpu

PATHS = {"two_kernel": 1, "cooperative": 2, "staged": 3}


def gpu_round(binding, x_np, d, alpha, lam, path):
    import torch
    M = x_np.shape[0]
    x = to_dev(x_np)
    norms = torch.full((M,), -1.0, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus(x, alpha, lam, norms_out=norms, ws=ws, d=d, path=path)
    assert binding.dppf_device_status(ws) == binding.OK
    return x.cpu().numpy(), norms.cpu().numpy()


def random_replicas(M, d, seed, base=0.02, drift=1e-3):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * base
    return padded((x0[None, :] + rng.standard_normal((M, d)) * drift).astype(np.float32))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 7, 8, 16, 17, 40, 100])
@pytest.mark.parametrize("d", [1, 3, 4, 31, 33, 127, 129, 4097, 100_003])
def test_small_shapes(oracle, M, d, path):
    _, binding = require_gpu()
    x = random_replicas(M, d, seed=M * 1000 + d)
    ref, r_ref = oracle.consensus(x, 0.1, 0.01, d=d)
    got, r = gpu_round(binding, x, d, 0.1, 0.01, PATHS[path])
    assert_parity(got, r, ref, r_ref, d)
    assert_pad_untouched(got, d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,d", [("C1", 1_048_576), ("C2", 3_000_017), ("C4", 5_000_005), ("C5", 2_000_003)])
def test_workload_recipes_scaled(oracle, name, d, path):
    """The benchmark recipes on vectors that span many tiles per block and a ragged tail."""
    _, binding = require_gpu()
    w = inputs.WORKLOADS[name].scaled(d)
    x = inputs.replicas(w)
    ref, r_ref = oracle.consensus(x, w.alpha, w.lam, d=w.d)
    got, r = gpu_round(binding, x, w.d, w.alpha, w.lam, PATHS[path])
    assert_parity(got, r, ref, r_ref, w.d)
    assert_pad_untouched(got, w.d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,d", [(129, 20_001), (300, 9_999), (1024, 30_003)])
def test_many_workers(oracle, M, d, path):
    """Worker counts far beyond the paper's (kernels with per-worker sums in shared memory)."""
    _, binding = require_gpu()
    x = random_replicas(M, d, seed=M)
    ref, r_ref = oracle.consensus(x, 0.1, 0.01, d=d)
    got, r = gpu_round(binding, x, d, 0.1, 0.01, PATHS[path])
    assert_parity(got, r, ref, r_ref, d)
    assert_pad_untouched(got, d)


@pytest.mark.parametrize("alpha,lam", [(1.0, 0.0), (0.5, 0.0), (0.0, 0.3), (0.9, 9.0), (0.5, 5.0), (0.05, 0.0)])
def test_invariant_parameter_corners(oracle, alpha, lam):
    _, binding = require_gpu()
    x = random_replicas(4, 70_001, seed=5, base=0.5, drift=0.1)
    ref, r_ref = oracle.consensus(x, alpha, lam, d=70_001)
    got, r = gpu_round(binding, x, 70_001, alpha, lam, 1)
    assert_parity(got, r, ref, r_ref, 70_001)
    if alpha == 0.0:     # push only: every replica moves by exactly lambda
        disp = np.linalg.norm(got[:, :70_001].astype(np.float64) - x[:, :70_001], axis=1)
        np.testing.assert_allclose(disp, np.float32(lam), rtol=1e-5)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 2, 3, 5, 16, 24])
def test_zero_distance_round_is_bit_exact(oracle, M, path):
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C5"].scaled(1_000_003)
    row = inputs.replicas(w, identical=True)[:1]
    row[0, [5, 4096, 999_999]] = np.float32(-0.0)       # unchanged means the sign of zeros too
    x = np.repeat(row, M, axis=0)
    ref, r_ref = oracle.consensus(x, w.alpha, w.lam, d=w.d)
    assert np.all(r_ref == 0.0) and same_bits(ref[:, :w.d], x[:, :w.d])
    got, r = gpu_round(binding, x, w.d, w.alpha, w.lam, PATHS[path])
    assert np.all(r == 0.0)
    assert same_bits(got[:, :w.d], x[:, :w.d])
    assert_pad_untouched(got, w.d)


def test_mixed_zero_and_nonzero_distances(oracle):
    """Two pairs of identical rows: no row is at zero distance, but deviations repeat exactly."""
    _, binding = require_gpu()
    base = random_replicas(2, 50_001, seed=9)
    x = np.ascontiguousarray(base[[0, 0, 1, 1]])
    ref, r_ref = oracle.consensus(x, 0.2, 0.05, d=50_001)
    got, r = gpu_round(binding, x, 50_001, 0.2, 0.05, 1)
    assert_parity(got, r, ref, r_ref, 50_001)
    assert same_bits(got[0, :50_001], got[1, :50_001]) and same_bits(got[2, :50_001], got[3, :50_001])


@pytest.mark.parametrize("M,d", [(4, 3_000_017), (8, 1_000_003), (16, 777_777), (20, 300_001), (64, 150_001)])
def test_reproducible_and_schedule_independent(M, d):
    """Same input -> same bits run to run for every schedule; the two register schedules
    also agree with each other bit for bit, the staged one to rounding of the distances."""
    _, binding = require_gpu()
    x = random_replicas(M, d, seed=11)
    a, ra = gpu_round(binding, x, d, 0.1, 0.01, 1)
    b, rb = gpu_round(binding, x, d, 0.1, 0.01, 1)
    c, rc = gpu_round(binding, x, d, 0.1, 0.01, 2)
    assert same_bits(a[:, :d], b[:, :d]) and same_bits(ra, rb)
    assert same_bits(a[:, :d], c[:, :d]) and same_bits(ra, rc)
    e, re_ = gpu_round(binding, x, d, 0.1, 0.01, 3)
    f, rf = gpu_round(binding, x, d, 0.1, 0.01, 3)
    assert same_bits(e[:, :d], f[:, :d]) and same_bits(re_, rf)
    np.testing.assert_allclose(re_, ra, rtol=2e-6)
    assert np.max(np.abs(e[:, :d].astype(np.float64) - a[:, :d])) <= 1e-8


@pytest.mark.parametrize("M,auto", [(4, 3), (8, 3), (16, 3), (20, 1)])
def test_the_schedule_that_ran_is_recorded(M, auto):
    """dppf_device_schedule reports what AUTO resolved to and what an explicit request ran."""
    _, binding = require_gpu()
    d = 300_001
    x = to_dev(random_replicas(M, d, seed=3))
    ws = binding.alloc_workspace(M, d)
    for path, want in ((0, auto), (1, 1), (2, 2 if M <= 16 else 1), (3, 3 if M <= 16 else 1)):
        binding.dppf_consensus(x, 0.1, 0.01, ws=ws, d=d, path=path)
        assert binding.dppf_device_schedule(ws) == want
    if M <= 16:
        binding.dppf_consensus_rounds(x, 0.1, 0.01, 3, ws=ws, d=d)
        assert binding.dppf_device_schedule(ws) == 3
        binding.dppf_consensus_general(x, 0.1, 0.01, ws=ws, d=d, path=1)
        assert binding.dppf_device_schedule(ws) == 1


@pytest.mark.parametrize("path", PATHS)
def test_resuming_from_a_saved_state_reproduces_the_run_bit_for_bit(path):
    """Checkpoint / resume: the state of the path is x (and v with the fused step); ten rounds in
    a row equal five rounds, a copy of the replicas through host memory into fresh buffers and a
    fresh workspace, and five more rounds."""
    import torch
    _, binding = require_gpu()
    d = 700_001
    w = inputs.WORKLOADS["C3"].scaled(d)
    x_np, v_np = random_replicas(4, d, seed=21), inputs.zeros_like_rows(w)
    g = to_dev(inputs.gradients(w, 0))

    def rounds(x, v, ws, k):
        for _ in range(k):
            binding.dppf_consensus(x, 0.1, 0.005, ws=ws, d=d, path=PATHS[path])
            binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay, 0.1, 0.005, ws=ws,
                                                  d=d, path=PATHS[path])

    xa, va = to_dev(x_np), to_dev(v_np)
    rounds(xa, va, binding.alloc_workspace(4, d), 10)
    xb, vb = to_dev(x_np), to_dev(v_np)
    rounds(xb, vb, binding.alloc_workspace(4, d), 5)
    saved_x, saved_v = xb.cpu().numpy().copy(), vb.cpu().numpy().copy()
    del xb, vb
    torch.cuda.empty_cache()
    xc, vc = to_dev(saved_x), to_dev(saved_v)
    rounds(xc, vc, binding.alloc_workspace(4, d), 5)
    assert same_bits(xa.cpu().numpy()[:, :d], xc.cpu().numpy()[:, :d])
    assert same_bits(va.cpu().numpy()[:, :d], vc.cpu().numpy()[:, :d])


def test_norms_out_is_optional_and_iterated_rounds_follow_oracle(oracle):
    import torch
    _, binding = require_gpu()
    d = 400_003
    x_np = random_replicas(4, d, seed=13)
    x = to_dev(x_np)
    ws = binding.alloc_workspace(4, d)
    ref = x_np
    for k in range(20):
        binding.dppf_consensus(x, 0.1, 0.005, norms_out=None, ws=ws, d=d, path=1 + k % 3)
        ref, r_ref = oracle.consensus(ref, 0.1, 0.005, d=d)
    norms = torch.zeros(4, device="cuda")
    binding.dppf_consensus(x, 0.1, 0.005, norms_out=norms, ws=ws, d=d)
    ref, r_ref = oracle.consensus(ref, 0.1, 0.005, d=d)
    assert_parity(x.cpu().numpy(), norms.cpu().numpy(), ref, r_ref, d)


def test_scheduled_rounds_follow_oracle_and_metrics():
    """Thirty rounds with the increasing push schedule; distances copied back each round feed
    the metric helper (mean distance, pull vs push strength)."""
    import torch
    import oracle
    oracle.build()
    _, binding = require_gpu()
    d, M, T, alpha, lam = 300_001, 4, 30, 0.1, 0.05
    x_np = random_replicas(M, d, seed=29)
    x = to_dev(x_np)
    ws = binding.alloc_workspace(M, d)
    norms = torch.zeros(M, device="cuda")
    ref = x_np
    for t in range(1, T + 1):
        lam_t = binding.dppf_lambda_schedule(binding.SCHEDULE_INCREASING, lam, t, T)
        binding.dppf_consensus(x, alpha, lam_t, norms_out=norms, ws=ws, d=d)
        ref, r_ref = oracle.consensus(ref, alpha, lam_t, d=d)
        mean, pull, push = binding.dppf_round_metrics(norms.cpu().tolist(), alpha, lam_t)
        assert abs(mean - r_ref.mean()) <= 1e-5 * r_ref.mean() and push == pytest.approx(lam_t)
        np.testing.assert_allclose(pull, np.float32(alpha) * r_ref, rtol=2e-5)
    assert_parity(x.cpu().numpy(), norms.cpu().numpy(), ref, r_ref, d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,d,tau", [(4, 1_000_003, 8), (2, 33, 3), (8, 200_001, 2), (16, 50_001, 2), (18, 40_003, 2), (1, 1000, 2)])
def test_local_steps_then_fused_round(oracle, M, d, tau, path):
    """tau-1 unfused local steps, then the last step fused with the round (x, v and r checked)."""
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C3"].scaled(d)
    w = type(w)(**{**w.__dict__, "M": M})
    x_np, v_np = inputs.replicas(w), inputs.zeros_like_rows(w)
    grads = [inputs.gradients(w, t) for t in range(tau)]
    ref_x, ref_v, r_ref = oracle.local_steps_then_consensus(
        x_np[:, :d], v_np[:, :d], [g[:, :d] for g in grads], w.lr, w.momentum, w.weight_decay, w.alpha, w.lam)
    x, v = to_dev(x_np), to_dev(v_np)
    ws = binding.alloc_workspace(M, d)
    norms = torch.zeros(M, device="cuda")
    for t in range(tau - 1):
        binding.dppf_local_step(x, v, to_dev(grads[t]), w.lr, w.momentum, w.weight_decay, d=d)
    g_last = to_dev(grads[-1])
    binding.dppf_local_step_and_consensus(x, v, g_last, w.lr, w.momentum, w.weight_decay, w.alpha, w.lam,
                                          norms_out=norms, ws=ws, d=d, path=PATHS[path])
    assert binding.dppf_device_status(ws) == binding.OK
    got_x, got_v = x.cpu().numpy(), v.cpu().numpy()
    assert_parity(got_x, norms.cpu().numpy(), ref_x, r_ref, d)
    verr = np.abs(got_v[:, :d].astype(np.float64) - ref_v[:, :d])
    assert np.all(verr <= 1e-6 * (1 + np.abs(ref_v[:, :d])))
    assert_pad_untouched(got_x, d), assert_pad_untouched(got_v, d)
    assert same_bits(g_last.cpu().numpy()[:, :d], grads[-1][:, :d])     # gradients are read-only


def test_random_shapes_fused_local_step(oracle):
    """Thirty seeded random cases of the fused local step + round over all schedules: worker
    counts 2..12 (the staged kernel up to 8, the register kernel above), ragged lengths, 1..3 steps."""
    import torch
    _, binding = require_gpu()
    rng = np.random.default_rng(20424_3)
    for case in range(30):
        M = int(rng.integers(2, 13))
        d = int(rng.choice([rng.integers(1, 9), rng.integers(9, 5000), rng.integers(5000, 300_000),
                            rng.integers(300_000, 1_200_000)]))
        tau = int(rng.integers(1, 4))
        path = int(rng.integers(1, 4))
        w = inputs.WORKLOADS["C3"].scaled(d)
        w = type(w)(**{**w.__dict__, "M": M})
        x_np, v_np = inputs.replicas(w, seed=9000 + case), inputs.zeros_like_rows(w)
        grads = [inputs.gradients(w, t, seed=9000 + case) for t in range(tau)]
        ref_x, ref_v, r_ref = oracle.local_steps_then_consensus(
            x_np[:, :d], v_np[:, :d], [g[:, :d] for g in grads], w.lr, w.momentum, w.weight_decay, w.alpha, w.lam)
        x, v = to_dev(x_np), to_dev(v_np)
        ws = binding.alloc_workspace(M, d)
        norms = torch.zeros(M, device="cuda")
        for t in range(tau - 1):
            binding.dppf_local_step(x, v, to_dev(grads[t]), w.lr, w.momentum, w.weight_decay, d=d)
        binding.dppf_local_step_and_consensus(x, v, to_dev(grads[-1]), w.lr, w.momentum, w.weight_decay, w.alpha,
                                              w.lam, norms_out=norms, ws=ws, d=d, path=path)
        assert binding.dppf_device_status(ws) == binding.OK
        info = f"case {case}: M={M} d={d} tau={tau} path={path}"
        got_x, got_v = x.cpu().numpy(), v.cpu().numpy()
        assert np.all(np.abs(norms.cpu().numpy() - r_ref) <= 1e-5 * r_ref), info
        err = np.abs(got_x[:, :d].astype(np.float64) - ref_x[:, :d])
        assert np.all(err <= 1e-6 * (1 + np.abs(ref_x[:, :d]))), f"{info}: max err {err.max():.3e}"
        verr = np.abs(got_v[:, :d].astype(np.float64) - ref_v[:, :d])
        assert np.all(verr <= 1e-6 * (1 + np.abs(ref_v[:, :d]))), info
        assert_pad_untouched(got_x, d), assert_pad_untouched(got_v, d)


def test_fused_matches_unfused_sequence():
    """Local step then round as two calls vs the fused call: the momentum buffers agree bit
    for bit (same arithmetic); the replicas agree to rounding of the distances (the two
    launches group the sum of squares into different per-block partials)."""
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C3"].scaled(3_000_001)
    x_np, v_np, g_np = inputs.replicas(w), inputs.zeros_like_rows(w), inputs.gradients(w, 0)
    x_np[:, :w.d] += inputs.gradients(w, 5)[:, :w.d]        # spread the replicas
    ws = binding.alloc_workspace(w.M, w.d)
    na, nb = torch.zeros(w.M, device="cuda"), torch.zeros(w.M, device="cuda")
    xa, va = to_dev(x_np), to_dev(v_np)
    binding.dppf_local_step(xa, va, to_dev(g_np), w.lr, w.momentum, w.weight_decay, d=w.d)
    binding.dppf_consensus(xa, w.alpha, w.lam, norms_out=na, ws=ws, d=w.d)
    xb, vb = to_dev(x_np), to_dev(v_np)
    binding.dppf_local_step_and_consensus(xb, vb, to_dev(g_np), w.lr, w.momentum, w.weight_decay,
                                          w.alpha, w.lam, norms_out=nb, ws=ws, d=w.d)
    assert same_bits(va.cpu().numpy()[:, :w.d], vb.cpu().numpy()[:, :w.d])
    np.testing.assert_allclose(nb.cpu().numpy(), na.cpu().numpy(), rtol=1e-6)
    xa_np, xb_np = xa.cpu().numpy()[:, :w.d], xb.cpu().numpy()[:, :w.d]
    assert np.max(np.abs(xa_np.astype(np.float64) - xb_np)) <= 1e-8


def test_host_resident_round(oracle):
    import torch
    _, binding = require_gpu()
    d = 500_003
    x_np = random_replicas(4, d, seed=17)
    ref, r_ref = oracle.consensus(x_np, 0.1, 0.01, d=d)
    x_host = torch.from_numpy(x_np.copy()).pin_memory()
    norms_host = torch.zeros(4).pin_memory()
    x_dev = binding.alloc_rows(4, d, fill=float("nan"))
    ws = binding.alloc_workspace(4, d)
    binding.dppf_consensus_host(x_host, 0.1, 0.01, norms_host, x_dev, ws, d=d)
    torch.cuda.synchronize()
    assert_parity(x_host.numpy(), norms_host.numpy(), ref, r_ref, d)
    assert_pad_untouched(x_host.numpy(), d)


def test_rounds_replayed_from_a_cuda_graph_match_eager_rounds():
    """dppf_consensus launches (cooperative kernels included) can be stream-captured once the
    first call on the device has been made; a replay gives the eager result bit for bit."""
    import torch
    _, binding = require_gpu()
    d = 1_000_003
    x_np = random_replicas(4, d, seed=37)
    ws = binding.alloc_workspace(4, d)
    norms = torch.zeros(4, device="cuda")
    eager = to_dev(x_np)
    for _ in range(5):
        binding.dppf_consensus(eager, 0.1, 0.005, norms_out=norms, ws=ws, d=d)
    eager_norms = norms.clone()
    x = to_dev(x_np)
    static = x.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(5):
            binding.dppf_consensus(static, 0.1, 0.005, norms_out=norms, ws=ws, d=d)
    static.copy_(x)
    graph.replay()
    torch.cuda.synchronize()
    assert same_bits(static.cpu().numpy()[:, :d], eager.cpu().numpy()[:, :d])
    assert torch.equal(norms, eager_norms)


def test_random_shapes_and_hyperparameters(oracle):
    """Eighty seeded random cases over the ranges the paper uses (alpha 0.05..0.9, lambda
    0.03..90, M 2..16) and a few beyond, every schedule, sizes that straddle tile and chunk
    boundaries."""
    _, binding = require_gpu()
    rng = np.random.default_rng(2507_20424)
    for case in range(80):
        M = int(rng.integers(2, 21))
        d = int(rng.choice([rng.integers(1, 64), rng.integers(64, 5000), rng.integers(5000, 400_000)]))
        alpha = float(rng.choice([0.05, 0.1, 0.3, 0.5, 0.9, 1.0]))
        lam = float(rng.choice([0.0, 0.03, 0.1, 0.5, 5.0, 9.0, 90.0]))
        base = float(rng.choice([0.02, 1.0, 30.0]))
        drift = base * float(rng.choice([1e-3, 5e-2, 1.0]))
        x = random_replicas(M, d, seed=1000 + case, base=base, drift=drift)
        path = int(rng.integers(1, 4))
        ref, r_ref = oracle.consensus(x, alpha, lam, d=d)
        got, r = gpu_round(binding, x, d, alpha, lam, path)
        # fp32 cannot do better than about one ulp of the largest operand (x_m or the step c_m dev_m):
        # with replicas far apart, or a push much longer than the distances, an updated element can be
        # much smaller than the terms it is formed from
        ref64 = ref[:, :d].astype(np.float64)
        err = np.abs(got[:, :d].astype(np.float64) - ref64)
        bound = 1e-6 * (1 + np.abs(ref64)) + 1.5e-7 * max(float(np.abs(x[:, :d]).max()), float(np.abs(ref64).max()))
        info = f"case {case}: M={M} d={d} alpha={alpha} lam={lam} base={base} drift={drift} path={path}"
        assert np.all(err <= bound), f"{info}: max err {err.max():.3e}"
        assert np.all(np.abs(r - r_ref) <= 1e-5 * r_ref), info
        if drift <= 0.05 * base and base <= 1.0 and lam <= 9.0:   # the regime of the workloads: stated tolerance as is
            assert_parity(got, r, ref, r_ref, d)
        assert_pad_untouched(got, d)


def test_host_resident_round_with_pageable_memory_and_no_norms(oracle):
    import torch
    _, binding = require_gpu()
    d = 123_457
    x_np = random_replicas(3, d, seed=43)
    ref, r_ref = oracle.consensus(x_np, 0.3, 0.02, d=d)
    x_host = torch.from_numpy(x_np.copy())                     # pageable: copies are staged by the driver
    x_dev = binding.alloc_rows(3, d, fill=float("nan"))
    ws = binding.alloc_workspace(3, d)
    binding.dppf_consensus_host(x_host, 0.3, 0.02, None, x_dev, ws, d=d)
    torch.cuda.synchronize()
    err = np.abs(x_host.numpy()[:, :d].astype(np.float64) - ref[:, :d])
    assert np.all(err <= 1e-6 * (1 + np.abs(ref[:, :d])))
    assert_pad_untouched(x_host.numpy(), d)


def test_runs_on_a_side_stream(oracle):
    import torch
    _, binding = require_gpu()
    d = 200_001
    x_np = random_replicas(3, d, seed=19)
    ref, r_ref = oracle.consensus(x_np, 0.3, 0.02, d=d)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        x = to_dev(x_np)
        norms = torch.zeros(3, device="cuda")
        binding.dppf_consensus(x, 0.3, 0.02, norms_out=norms, d=d)
    s.synchronize()
    assert_parity(x.cpu().numpy(), norms.cpu().numpy(), ref, r_ref, d)


def test_calls_on_two_streams_with_their_own_workspaces_do_not_interfere(oracle):
    """Two independent replica sets, each with its own workspace, driven from two streams at once
    (cooperative launches of the two take turns on the GPU): both match the oracle."""
    import torch
    _, binding = require_gpu()
    d = 1_500_003
    xs_np = [random_replicas(4, d, seed=51), random_replicas(8, d, seed=52)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    xs, norms, wss = [], [], []
    for x_np in xs_np:
        xs.append(to_dev(x_np))
        norms.append(torch.zeros(3, x_np.shape[0], device="cuda"))
        wss.append(binding.alloc_workspace(x_np.shape[0], d))
    torch.cuda.synchronize()
    for rep in range(3):
        for i, s in enumerate(streams):
            with torch.cuda.stream(s):
                binding.dppf_consensus(xs[i], 0.1, 0.01, norms_out=norms[i][rep], ws=wss[i], d=d)
    for s in streams:
        s.synchronize()
    for i, x_np in enumerate(xs_np):
        ref = x_np
        for rep in range(3):
            ref, r_ref = oracle.consensus(ref, 0.1, 0.01, d=d)
            assert np.all(np.abs(norms[i][rep].cpu().numpy() - r_ref) <= 1e-5 * r_ref)
        assert_parity(xs[i].cpu().numpy(), norms[i][2].cpu().numpy(), ref, r_ref, d)
