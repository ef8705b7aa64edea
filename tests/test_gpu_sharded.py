"""A round split at its reduction (column shards, one per GPU in a multi-GPU run): the distance
pass per shard, the M sums of squares added over the shards, the update pass per shard.  Here
the shards are column ranges of one buffer on one GPU and the sums are added on the device; the
result must be the oracle's round on the whole vector."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, padded, require_gpu, same_bits, to_dev

pytestmark = pytest.mark.gpu


def replicas(M, d, seed):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * 0.02
    return padded((x0[None, :] + rng.standard_normal((M, d)) * 1e-3).astype(np.float32))


def sharded_round(binding, x, d, cuts, alpha, lam):
    """x: [M, ld] CUDA tensor; cuts: shard boundaries (multiples of 32 columns)."""
    import torch
    M = x.shape[0]
    bounds = [0, *cuts, d]
    total = torch.zeros(M, dtype=torch.float64, device="cuda")
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        part = torch.full((M,), -1.0, dtype=torch.float64, device="cuda")
        binding.dppf_distance_partials(x[:, lo:], part, d=hi - lo)
        total += part                                    # the exchange: M doubles per shard
    norms = torch.zeros(M, device="cuda")
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        binding.dppf_update_from_sums(x[:, lo:], alpha, lam, total, norms_out=norms, d=hi - lo)
    torch.cuda.synchronize()
    return norms


@pytest.mark.parametrize("M,d,cuts", [(4, 3_000_017, [1_500_000 // 32 * 32]), (8, 1_000_003, [320_000, 640_000]),
                                      (16, 500_001, [250_016]), (2, 100, [32, 64]), (24, 200_003, [100_000 // 32 * 32]),
                                      (1, 5000, [2528])])
def test_column_shards_reproduce_the_round_on_the_whole_vector(oracle, M, d, cuts):
    _, binding = require_gpu()
    x_np = replicas(M, d, seed=M + len(cuts))
    ref, r_ref = oracle.consensus(x_np, 0.1, 0.01, d=d)
    x = to_dev(x_np)
    norms = sharded_round(binding, x, d, cuts, 0.1, 0.01)
    got = x.cpu().numpy()
    assert_parity(got, norms.cpu().numpy(), ref, r_ref, d)
    assert_pad_untouched(got, d)


def test_one_shard_is_the_two_launch_round_bit_for_bit():
    import torch
    _, binding = require_gpu()
    d = 2_000_003
    x_np = replicas(4, d, seed=3)
    xa, xb = to_dev(x_np), to_dev(x_np)
    na = torch.zeros(4, device="cuda")
    binding.dppf_consensus(xa, 0.1, 0.01, norms_out=na, d=d, path=1)
    nb = sharded_round(binding, xb, d, [], 0.1, 0.01)
    assert same_bits(xa.cpu().numpy()[:, :d], xb.cpu().numpy()[:, :d]) and torch.equal(na, nb)


def test_identical_replicas_and_bad_arguments():
    import torch
    _, binding = require_gpu()
    d = 100_003
    row = replicas(1, d, 5)
    x_np = np.repeat(row, 3, axis=0)
    x = to_dev(x_np)
    norms = sharded_round(binding, x, d, [50_016], 0.2, 0.05)
    assert same_bits(x.cpu().numpy()[:, :d], x_np[:, :d]) and torch.all(norms == 0)
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")
    lib = binding.load()
    assert lib.dppf_distance_partials(x.data_ptr(), 3, d, x.stride(0), None, 0x10000000, 1 << 30, None) == binding.ERR_INVALID_ARG
    assert lib.dppf_update_from_sums(x.data_ptr(), 3, d, x.stride(0), float("nan"), 0.1, sums.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert lib.dppf_update_from_sums(x.data_ptr() + 4, 3, d, x.stride(0), 0.1, 0.1, sums.data_ptr(), None, None) == binding.ERR_ALIGNMENT
