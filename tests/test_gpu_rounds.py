"""Several rounds in one launch (dppf_consensus_rounds) vs the CPU oracle iterated the same
number of times, through the C ABI: the replicas after the last round and the distances
before every round."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev
from paper_2507_20424_b200 import inputs

pytestmark = pytest.mark.gpu

PATHS = {"two_kernel": 1, "register": 2, "staged": 3}


def replicas(M, d, seed, base=0.02, drift=1e-3):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * base
    return padded((x0[None, :] + rng.standard_normal((M, d)) * drift).astype(np.float32))


def oracle_rounds(oracle, x, alpha, lams, d):
    """The oracle's round applied len(lams) times; returns the last state and every round's r."""
    rs = []
    for lam in lams:
        x, r = oracle.consensus(x, alpha, lam, d=d)
        rs.append(r)
    return x, np.array(rs)


def gpu_rounds(binding, x_np, d, alpha, lam, n, path, lambdas=None):
    import torch
    M = x_np.shape[0]
    x = to_dev(x_np)
    norms = torch.full((n, M), -1.0, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus_rounds(x, alpha, lam, n, lambdas=lambdas, norms_out=norms, ws=ws, d=d, path=path)
    assert binding.dppf_device_status(ws) == binding.OK
    return x.cpu().numpy(), norms.cpu().numpy()


def check(got, norms, ref, rs, d):
    assert_parity(got, norms[-1], ref, rs[-1], d)
    assert np.all(np.abs(norms - rs) <= 1e-5 * rs), (norms, rs)
    assert np.all(norms[rs == 0.0] == 0.0)
    assert_pad_untouched(got, d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("n", [1, 2, 3, 8])
@pytest.mark.parametrize("M,d", [(2, 5), (3, 4099), (4, 1_000_003), (4, 3_000_017), (5, 70_003), (8, 2_400_001),
                                 (9, 300_001), (16, 777_777), (1, 1000), (20, 50_001)])
def test_rounds_match_the_iterated_oracle(oracle, M, d, n, path):
    _, binding = require_gpu()
    x = replicas(M, d, seed=M * 131 + d % 89 + n)
    ref, rs = oracle_rounds(oracle, x, 0.1, [0.01] * n, d)
    got, norms = gpu_rounds(binding, x, d, 0.1, 0.01, n, PATHS[path])
    check(got, norms, ref, rs, d)


@pytest.mark.parametrize("path", ["register", "staged"])
def test_push_schedule_per_round(oracle, path):
    """The increasing cosine push schedule over 30 rounds in one call."""
    _, binding = require_gpu()
    M, d, T, alpha, lam = 4, 1_500_001, 30, 0.1, 0.05
    x = replicas(M, d, seed=29)
    lams = [binding.dppf_lambda_schedule(binding.SCHEDULE_INCREASING, lam, t, T) for t in range(1, T + 1)]
    ref, rs = oracle_rounds(oracle, x, alpha, lams, d)
    got, norms = gpu_rounds(binding, x, d, alpha, 123.0, T, PATHS[path], lambdas=lams)   # `lam` ignored
    check(got, norms, ref, rs, d)


@pytest.mark.parametrize("path", ["register", "staged"])
def test_more_rounds_than_one_launch_holds(oracle, path):
    """600 rounds: three launches; the distances settle at lambda / alpha (Theorem 1)."""
    _, binding = require_gpu()
    M, d, n, alpha, lam = 4, 40_003, 600, 0.1, 0.005
    x = replicas(M, d, seed=31)
    ref, rs = oracle_rounds(oracle, x, alpha, [lam] * n, d)
    got, norms = gpu_rounds(binding, x, d, alpha, lam, n, PATHS[path])
    check(got, norms, ref, rs, d)
    np.testing.assert_allclose(norms[-1], np.float32(lam) / np.float32(alpha), rtol=1e-3)


@pytest.mark.parametrize("M,d", [(4, 5_000_005), (8, 1_000_003), (16, 1_200_001)])
def test_reproducible_and_close_to_single_calls(M, d):
    """Same input -> same bits run to run; n single calls give the same replicas up to the
    rounding of the distances (their sums of squares are grouped differently)."""
    import torch
    _, binding = require_gpu()
    x = replicas(M, d, seed=11)
    for path in (2, 3):
        a, ra = gpu_rounds(binding, x, d, 0.1, 0.01, 5, path)
        b, rb = gpu_rounds(binding, x, d, 0.1, 0.01, 5, path)
        assert same_bits(a[:, :d], b[:, :d]) and same_bits(ra, rb)
        xs = to_dev(x)
        ns = torch.zeros(M, device="cuda")
        ws = binding.alloc_workspace(M, d)
        singles = []
        for _ in range(5):
            binding.dppf_consensus(xs, 0.1, 0.01, norms_out=ns, ws=ws, d=d)
            singles.append(ns.cpu().numpy())
        np.testing.assert_allclose(ra, np.array(singles), rtol=5e-6)
        assert np.max(np.abs(a[:, :d].astype(np.float64) - xs.cpu().numpy()[:, :d])) <= 2e-8


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 3, 16])
def test_identical_replicas_stay_untouched_over_rounds(M, path):
    _, binding = require_gpu()
    row = replicas(1, 300_003, 5)
    row[0, [0, 77, 300_002]] = np.float32(-0.0)
    x = np.repeat(row, M, axis=0)
    got, norms = gpu_rounds(binding, x, 300_003, 0.2, 0.05, 4, PATHS[path])
    assert same_bits(got[:, :300_003], x[:, :300_003]) and np.all(norms == 0.0)


def test_norms_out_is_optional_and_bad_arguments_are_refused():
    import torch
    _, binding = require_gpu()
    d = 200_001
    x_np = replicas(4, d, 3)
    a, _ = gpu_rounds(binding, x_np, d, 0.1, 0.01, 3, 0)
    x = to_dev(x_np)
    binding.dppf_consensus_rounds(x, 0.1, 0.01, 3, d=d)
    torch.cuda.synchronize()
    assert same_bits(x.cpu().numpy()[:, :d], a[:, :d])
    for kwargs in (dict(n_rounds=0), dict(n_rounds=2, lambdas=[0.1, float("inf")])):
        with pytest.raises(binding.DppfError) as e:
            binding.dppf_consensus_rounds(x, 0.1, 0.01, d=d, **kwargs)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DppfError):
        binding.dppf_consensus_rounds(x, float("nan"), 0.01, 2, d=d)
    torch.cuda.synchronize()
    assert same_bits(x.cpu().numpy()[:, :d], a[:, :d])


def test_random_shapes_rounds_and_schedules(oracle):
    """Forty seeded random cases: worker counts 2..16, vector lengths that straddle the tail
    columns, one chunk, one ring and several rings per block, 1..6 rounds, every schedule."""
    _, binding = require_gpu()
    rng = np.random.default_rng(20424_7)
    for case in range(40):
        M = int(rng.integers(2, 17))
        d = int(rng.choice([rng.integers(1, 9), rng.integers(9, 5000), rng.integers(5000, 400_000),
                            rng.integers(400_000, 1_500_000)]))
        n = int(rng.integers(1, 7))
        alpha = float(rng.choice([0.05, 0.1, 0.5, 0.9]))
        lam = float(rng.choice([0.0, 0.01, 0.05, 0.5]))
        if lam == 0.0:
            alpha = min(alpha, 0.1)     # a strong pull with no push collapses the replicas to within a few
                                        # fp32 ulps of each other, where no distance has five good digits
        path = int(rng.integers(1, 4))
        x = replicas(M, d, seed=5000 + case)
        ref, rs = oracle_rounds(oracle, x, alpha, [lam] * n, d)
        got, norms = gpu_rounds(binding, x, d, alpha, lam, n, path)
        info = f"case {case}: M={M} d={d} n={n} alpha={alpha} lam={lam} path={path}"
        assert np.all(np.abs(norms - rs) <= 1e-5 * rs), info
        err = np.abs(got[:, :d].astype(np.float64) - ref[:, :d])
        assert np.all(err <= 1e-6 * (1 + np.abs(ref[:, :d]))), f"{info}: max err {err.max():.3e}"
        assert_pad_untouched(got, d)


def test_rounds_call_replayed_from_a_cuda_graph():
    """Once the first call on the device has been made, a multi-round call can be stream-captured;
    the replay gives the eager result bit for bit."""
    import torch
    _, binding = require_gpu()
    d = 1_000_003
    x_np = replicas(4, d, seed=37)
    ws = binding.alloc_workspace(4, d)
    norms = torch.zeros(6, 4, device="cuda")
    eager = to_dev(x_np)
    binding.dppf_consensus_rounds(eager, 0.1, 0.005, 6, norms_out=norms, ws=ws, d=d)
    eager_norms = norms.clone()
    x = to_dev(x_np)
    static = x.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.dppf_consensus_rounds(static, 0.1, 0.005, 6, norms_out=norms, ws=ws, d=d)
    static.copy_(x)
    graph.replay()
    torch.cuda.synchronize()
    assert same_bits(static.cpu().numpy()[:, :d], eager.cpu().numpy()[:, :d])
    assert torch.equal(norms, eager_norms)


@pytest.mark.parametrize("M,path", [(4, 3), (8, 3), (3, 2), (16, 3)])
def test_distances_follow_the_closed_form_of_theorem_1(M, path):
    """No oracle involved: on a centred regular simplex the unit directions sum to zero, so the
    average never moves and every distance obeys r_k = lambda/alpha + (1-alpha)^k (r_0 - lambda/alpha)
    (proof of Theorem 1); with lambda = 0.5, alpha = 0.1 it settles at the 5 the paper prints."""
    import torch
    _, binding = require_gpu()
    d, n, alpha, lam, r0 = 120_000 // M * M, 60, 0.1, 0.5, 2.0
    block = d // M
    e = np.zeros((M, d))
    for m in range(M):
        e[m, m * block:(m + 1) * block] = 1.0 / np.sqrt(block)        # orthonormal rows
    centred = e - e.mean(axis=0)
    centred *= r0 / np.linalg.norm(centred[0])
    x_np = padded((0.3 + centred).astype(np.float32))
    x = to_dev(x_np)
    norms = torch.zeros(n, M, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus_rounds(x, alpha, lam, n, norms_out=norms, ws=ws, d=d, path=path)
    assert binding.dppf_device_status(ws) == binding.OK
    r = norms.cpu().numpy().astype(np.float64)
    a32, l32 = float(np.float32(alpha)), float(np.float32(lam))
    r_start = np.linalg.norm(x_np[:, :d].astype(np.float64) - x_np[:, :d].astype(np.float64).mean(axis=0), axis=1)
    k = np.arange(n)[:, None]
    want = l32 / a32 + (1.0 - a32) ** k * (r_start[None, :] - l32 / a32)
    np.testing.assert_allclose(r, want, rtol=2e-5)
    assert abs(want[-1, 0] - 5.0) < 0.01                               # 5 = lambda / alpha
    mean_after = x.cpu().numpy()[:, :d].astype(np.float64).mean(axis=0)
    np.testing.assert_allclose(mean_after, x_np[:, :d].astype(np.float64).mean(axis=0), atol=2e-6)
