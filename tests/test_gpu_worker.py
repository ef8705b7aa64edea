"""One replica per GPU (the paper's own deployment): each worker's pull-push update from the
all-reduced parameters, against the CPU oracle.  The collective is stood in for by a sum over
the rows on the device, which is all an all-reduce would hand to the call."""
import numpy as np
import pytest

from gpu_util import require_gpu, same_bits

pytestmark = pytest.mark.gpu


def replicas(M, d, seed):
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(d) * 0.02
    return (x0[None, :] + rng.standard_normal((M, d)) * 1e-3).astype(np.float32)


@pytest.mark.parametrize("M,d", [(4, 3_000_017), (8, 1_000_003), (3, 4099), (2, 5), (5, 70_001), (16, 300_000)])
@pytest.mark.parametrize("mean", [False, True])
def test_every_worker_matches_the_oracle_and_the_round(oracle, M, d, mean):
    import torch
    _, binding = require_gpu()
    x_np = replicas(M, d, seed=M + d % 13)
    xs = torch.from_numpy(x_np).cuda()
    reduced = xs.sum(dim=0)                       # what a sum all-reduce leaves on every GPU
    scale = 1.0 / M
    if mean:
        reduced, scale = reduced / M, 1.0
    red_np = reduced.cpu().numpy()
    ref_round, r_round = oracle.consensus(x_np, 0.1, 0.01)
    norm = torch.zeros(1, device="cuda")
    for m in range(M):
        x = xs[m].clone()
        ws = binding.dppf_worker_update(x, reduced, scale, 0.1, 0.01, norm_out=norm)
        assert binding.dppf_device_status(ws) == binding.OK
        want, r = oracle.worker_update(x_np[m], red_np, scale, 0.1, 0.01)
        got = x.cpu().numpy()
        assert abs(float(norm.item()) - r) <= 1e-5 * r
        err = np.abs(got.astype(np.float64) - want)
        assert np.all(err <= 1e-6 * (1 + np.abs(want))), float(err.max())
        # and, through the fp32 average, the same replica the one-GPU round produces
        assert abs(float(norm.item()) - r_round[m]) <= 1e-5 * r_round[m]
        assert np.all(np.abs(got.astype(np.float64) - ref_round[m]) <= 1e-6 * (1 + np.abs(ref_round[m])))


def test_worker_on_the_average_is_untouched_and_bad_arguments_are_refused():
    import torch
    _, binding = require_gpu()
    d = 100_003
    x_np = replicas(1, d, 3)[0]
    x_np[[0, 17]] = np.float32(-0.0)
    x = torch.from_numpy(x_np).cuda()
    reduced = x.clone() * 4
    norm = torch.ones(1, device="cuda")
    binding.dppf_worker_update(x, reduced, 0.25, 0.2, 0.05, norm_out=norm)
    torch.cuda.synchronize()
    assert same_bits(x.cpu().numpy(), x_np) and float(norm.item()) == 0.0
    lib = binding.load()
    ws = binding.alloc_workspace(1, d)
    args = (x.data_ptr(), reduced.data_ptr(), 0.25, d, 0.1, 0.01, None, ws.data_ptr(), ws.numel(), None)
    assert lib.dppf_worker_update(*args) == binding.OK
    assert lib.dppf_worker_update(args[0], None, *args[2:]) == binding.ERR_INVALID_ARG
    assert lib.dppf_worker_update(args[0], args[0], *args[2:]) == binding.ERR_INVALID_ARG          # aliases x
    assert lib.dppf_worker_update(args[0], args[1] + 4, *args[2:]) == binding.ERR_ALIGNMENT
    assert lib.dppf_worker_update(args[0], args[1], float("nan"), *args[3:]) == binding.ERR_INVALID_ARG
    assert lib.dppf_worker_update(*args[:8], 16, None) == binding.ERR_WORKSPACE
    torch.cuda.synchronize()


def test_reproducible_run_to_run():
    import torch
    _, binding = require_gpu()
    d = 2_000_003
    x_np = replicas(4, d, 9)
    xs = torch.from_numpy(x_np).cuda()
    reduced = xs.sum(dim=0)
    outs = []
    for _ in range(2):
        x = xs[1].clone()
        n = torch.zeros(1, device="cuda")
        binding.dppf_worker_update(x, reduced, 0.25, 0.1, 0.005, norm_out=n)
        outs.append((x.cpu().numpy(), n.cpu().numpy()))
    assert same_bits(outs[0][0], outs[1][0]) and same_bits(outs[0][1], outs[1][1])
