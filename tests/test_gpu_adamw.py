"""AdamW as the local optimiser (the paper's ViT setting): stand-alone steps and the last
step fused with the round, on the GPU vs the fp64 oracle."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, require_gpu, same_bits, to_dev
from paper_2507_20424_b200 import inputs

pytestmark = pytest.mark.gpu

HP = dict(lr=5e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)      # ViT runs of the paper


def workload(M, d):
    w = inputs.WORKLOADS["C3"].scaled(d)
    return type(w)(**{**w.__dict__, "M": M, "alpha": 0.9, "lam": 0.09})


def close(got, ref):
    """Moment buffers: fp32 rounding of terms as large as the largest entry, plus 1e-5 relative."""
    ref = np.asarray(ref, dtype=np.float64)
    return np.all(np.abs(got.astype(np.float64) - ref) <= 2e-6 * np.abs(ref).max() + 1e-5 * np.abs(ref))


@pytest.mark.parametrize("path", [2, 1])          # one cooperative launch / two launches
@pytest.mark.parametrize("M,d,tau", [(1, 1003, 2), (2, 33, 3), (4, 1_000_003, 4), (8, 200_001, 2), (16, 50_001, 2), (5, 7, 1),
                                     (7, 300_001, 2), (12, 150_003, 2)])
def test_adamw_steps_then_fused_round(oracle, M, d, tau, path):
    import torch
    _, binding = require_gpu()
    w = workload(M, d)
    x_np = inputs.replicas(w)
    a_np, b_np = inputs.zeros_like_rows(w), inputs.zeros_like_rows(w)
    grads = [inputs.gradients(w, t) for t in range(tau)]
    x64, a64, b64 = oracle.adamw_steps_f64(x_np[:, :d], a_np[:, :d], b_np[:, :d], [g[:, :d] for g in grads], **HP)
    ref, r_ref = oracle.consensus_f64(x64, w.alpha, w.lam)
    x, a, b = to_dev(x_np), to_dev(a_np), to_dev(b_np)
    norms = torch.zeros(M, device="cuda")
    ws = binding.alloc_workspace(M, d)
    for t in range(tau - 1):
        binding.dppf_adamw_step(x, a, b, to_dev(grads[t]), step=t + 1, d=d, **HP)
    g_last = to_dev(grads[-1])
    binding.dppf_adamw_step_and_consensus(x, a, b, g_last, step=tau, alpha=w.alpha, lam=w.lam,
                                          norms_out=norms, ws=ws, d=d, path=path, **HP)
    assert binding.dppf_device_status(ws) == binding.OK
    got_x, got_a, got_b = x.cpu().numpy(), a.cpu().numpy(), b.cpu().numpy()
    assert_parity(got_x, norms.cpu().numpy(), ref, r_ref, d)
    assert close(got_a[:, :d], a64) and close(got_b[:, :d], b64)
    for arr in (got_x, got_a, got_b):
        assert_pad_untouched(arr, d)
    assert same_bits(g_last.cpu().numpy()[:, :d], grads[-1][:, :d])


def test_fused_matches_step_then_round():
    import torch
    _, binding = require_gpu()
    w = workload(4, 2_000_003)
    x_np, z = inputs.replicas(w), inputs.zeros_like_rows(w)
    x_np[:, :w.d] += inputs.gradients(w, 7)[:, :w.d]
    g = inputs.gradients(w, 0)
    xa, aa, ba = to_dev(x_np), to_dev(z), to_dev(z)
    binding.dppf_adamw_step(xa, aa, ba, to_dev(g), step=1, d=w.d, **HP)
    na = torch.zeros(4, device="cuda")
    binding.dppf_consensus(xa, w.alpha, w.lam, norms_out=na, d=w.d)
    xb, ab, bb = to_dev(x_np), to_dev(z), to_dev(z)
    nb = torch.zeros(4, device="cuda")
    binding.dppf_adamw_step_and_consensus(xb, ab, bb, to_dev(g), step=1, alpha=w.alpha, lam=w.lam, norms_out=nb,
                                          d=w.d, **HP)
    assert same_bits(aa.cpu().numpy()[:, :w.d], ab.cpu().numpy()[:, :w.d])
    assert same_bits(ba.cpu().numpy()[:, :w.d], bb.cpu().numpy()[:, :w.d])
    np.testing.assert_allclose(nb.cpu().numpy(), na.cpu().numpy(), rtol=2e-6)
    assert np.max(np.abs(xa.cpu().numpy()[:, :w.d].astype(np.float64) - xb.cpu().numpy()[:, :w.d])) <= 1e-7


@pytest.mark.parametrize("M", [4, 8, 16])
def test_both_schedules_agree_bit_for_bit(M):
    import torch
    _, binding = require_gpu()
    w = workload(M, 1_200_003)
    x_np, z, g = inputs.replicas(w), inputs.zeros_like_rows(w), inputs.gradients(w, 0)
    x_np[:, :w.d] += inputs.gradients(w, 7)[:, :w.d]
    outs = []
    for path in (2, 1):
        x, a, b = to_dev(x_np), to_dev(z), to_dev(z)
        n = torch.zeros(M, device="cuda")
        binding.dppf_adamw_step_and_consensus(x, a, b, to_dev(g), step=3, alpha=w.alpha, lam=w.lam, norms_out=n,
                                              d=w.d, path=path, **HP)
        outs.append((x.cpu().numpy()[:, :w.d], a.cpu().numpy()[:, :w.d], b.cpu().numpy()[:, :w.d], n.cpu().numpy()))
    assert all(same_bits(p, q) for p, q in zip(*outs))


def test_adamw_rejects_bad_arguments():
    _, binding = require_gpu()
    w = workload(2, 1000)
    x, a, b, g = (to_dev(inputs.zeros_like_rows(w)) for _ in range(4))
    for bad in (dict(step=0), dict(beta1=1.0), dict(beta2=-0.1), dict(lr=float("nan"))):
        kw = {**HP, "step": 1, **bad}
        with pytest.raises(binding.DppfError) as e:
            binding.dppf_adamw_step(x, a, b, g, d=1000, **kw)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DppfError):
        binding.dppf_adamw_step(x, x, b, g, step=1, d=1000, **HP)
