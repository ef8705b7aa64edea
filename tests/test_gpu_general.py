"""General round (arbitrary consensus variable, push from x_A or x_C, optional second
gradient term) on the GPU vs the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev
from paper_2507_20424_b200 import inputs

pytestmark = pytest.mark.gpu


def replicas(M, d, seed, base=0.02, drift=1e-3):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * base
    return padded((x0[None, :] + rng.standard_normal((M, d)) * drift).astype(np.float32))


PATHS = {"staged": 3, "two_kernel": 1}


def run(binding, x_np, d, alpha, lam, weights, push_from, two_term, path=0):
    import torch
    M = x_np.shape[0]
    x = to_dev(x_np)
    r = torch.full((M,), -1.0, device="cuda")
    n = torch.full((M,), -1.0, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus_general(x, alpha, lam, weights,
                                   {"average": 0, "consensus": 1}[push_from], two_term,
                                   norms_out=r, push_norms_out=n, ws=ws, d=d, path=path)
    assert binding.dppf_device_status(ws) == binding.OK
    return x.cpu().numpy(), r.cpu().numpy(), n.cpu().numpy()


def weights_for(kind, M, seed):
    if kind == "none":
        return None
    if kind == "leader":
        w = np.zeros(M)
        w[seed % M] = 1.0
        return w
    return np.random.default_rng(seed).random(M) + 0.05


def check(got, r, n, ref, r_ref, n_ref, d):
    assert_parity(got, r, ref, r_ref, d)
    assert np.all(np.abs(n - n_ref) <= 1e-5 * n_ref + 1e-30)
    assert np.all(n[n_ref == 0.0] == 0.0)
    assert_pad_untouched(got, d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("two_term", [False, True])
@pytest.mark.parametrize("push_from", ["average", "consensus"])
@pytest.mark.parametrize("wkind", ["none", "random", "leader"])
@pytest.mark.parametrize("M,d", [(1, 1000), (2, 5), (3, 4099), (4, 300_001), (5, 70_003), (8, 1_000_003),
                                 (16, 200_001)])
def test_general_round_matches_oracle(oracle, M, d, wkind, push_from, two_term, path):
    _, binding = require_gpu()
    x = replicas(M, d, seed=M * 31 + d % 97)
    w = weights_for(wkind, M, d)
    ref, r_ref, n_ref = oracle.consensus_general(x, 0.1, 0.01, w, push_from, two_term, d=d)
    got, r, n = run(binding, x, d, 0.1, 0.01, w, push_from, two_term, PATHS[path])
    check(got, r, n, ref, r_ref, n_ref, d)


@pytest.mark.parametrize("wkind,push_from,two_term", [("random", "consensus", True), ("leader", "consensus", False),
                                                      ("random", "average", True), ("leader", "average", True)])
@pytest.mark.parametrize("M,d", [(4, 5_000_005), (8, 3_000_017), (12, 2_000_003), (16, 1_500_001)])
def test_weighted_rounds_with_more_chunks_per_block_than_ring_stages(oracle, M, d, wkind, push_from, two_term):
    """Vectors long enough that every block wraps its ring several times in the distance pass and
    refills stages in the update pass, with every flavour of the arithmetic."""
    _, binding = require_gpu()
    x = replicas(M, d, seed=M + d % 101)
    w = weights_for(wkind, M, 3)
    ref, r_ref, n_ref = oracle.consensus_general(x, 0.1, 0.02, w, push_from, two_term, d=d)
    got, r, n = run(binding, x, d, 0.1, 0.02, w, push_from, two_term, 3)
    check(got, r, n, ref, r_ref, n_ref, d)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("weights", [None, [2.0, 2.0, 2.0, 2.0]])
def test_hard_consensus_with_equal_weights_collapses_onto_the_average(oracle, path, weights):
    """alpha = 1 (the DDP / hard-consensus case of Algorithm 1) with the push taken from the
    average: every pulled point IS the average, so no worker has a push direction; the
    replicas collapse onto x_A and the push distances are exactly zero, whatever lambda is."""
    _, binding = require_gpu()
    d = 400_003
    x = replicas(4, d, seed=71)
    ref, r_ref, n_ref = oracle.consensus_general(x, 1.0, 0.5, weights, "average", False, d=d)
    assert np.all(n_ref == 0.0)
    got, r, n = run(binding, x, d, 1.0, 0.5, weights, "average", False, PATHS[path])
    assert np.all(n == 0.0)
    check(got, r, n, ref, r_ref, n_ref, d)
    spread = np.abs(got[:, :d].astype(np.float64) - got[0, :d]).max()        # all on x_A, to fp32 rounding
    assert spread <= 4e-9


def test_defaults_agree_with_the_plain_round(oracle):
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C2"].scaled(3_000_017)
    x_np = inputs.replicas(w)
    got, r, n = run(binding, x_np, w.d, w.alpha, w.lam, None, "average", False)
    xa = to_dev(x_np)
    na = torch.zeros(w.M, device="cuda")
    binding.dppf_consensus(xa, w.alpha, w.lam, norms_out=na, d=w.d)
    np.testing.assert_allclose(r, na.cpu().numpy(), rtol=2e-6)
    assert np.max(np.abs(got[:, :w.d].astype(np.float64) - xa.cpu().numpy()[:, :w.d])) <= 1e-7
    ref, r_ref = oracle.consensus(x_np, w.alpha, w.lam, d=w.d)
    assert_parity(got, r, ref, r_ref, w.d)


def test_second_term_keeps_the_average_on_the_gpu():
    _, binding = require_gpu()
    x = replicas(8, 500_003, 77, base=0.05, drift=5e-3)
    d = 500_003
    got, _, _ = run(binding, x, d, 0.05, 0.02, None, "average", True)
    np.testing.assert_allclose(got[:, :d].astype(np.float64).mean(axis=0), x[:, :d].astype(np.float64).mean(axis=0),
                               rtol=0, atol=2e-8)


@pytest.mark.parametrize("M", [1, 3, 16])
def test_identical_replicas_are_not_touched(M):
    _, binding = require_gpu()
    row = replicas(1, 100_003, 5)
    row[0, [0, 77, 100_002]] = np.float32(-0.0)
    x = np.repeat(row, M, axis=0)
    got, r, n = run(binding, x, 100_003, 0.2, 0.05, list(range(1, M + 1)), "consensus", True)
    assert same_bits(got[:, :100_003], x[:, :100_003]) and np.all(r == 0) and np.all(n == 0)


def test_reproducible_and_rejects_bad_arguments():
    import torch
    _, binding = require_gpu()
    x = replicas(4, 1_000_003, 9)
    a = run(binding, x, 1_000_003, 0.1, 0.01, [1, 2, 3, 4], "consensus", True)
    b = run(binding, x, 1_000_003, 0.1, 0.01, [1, 2, 3, 4], "consensus", True)
    assert all(same_bits(p, q) for p, q in zip(a, b))
    xd = to_dev(x)
    for kwargs in (dict(weights=[0, 0, 0, 0]), dict(weights=[1, float("nan"), 1, 1]), dict(push_from=5)):
        with pytest.raises(binding.DppfError) as e:
            binding.dppf_consensus_general(xd, 0.1, 0.01, d=1_000_003, **kwargs)
        assert e.value.status == binding.ERR_INVALID_ARG
    x17 = to_dev(replicas(17, 100, 3))
    with pytest.raises(binding.DppfError):
        binding.dppf_consensus_general(x17, 0.1, 0.01, d=100)
    torch.cuda.synchronize()
    assert same_bits(xd.cpu().numpy()[:, :1_000_003], x[:, :1_000_003])
