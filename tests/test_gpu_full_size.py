"""The five benchmark workloads at their full sizes, in the launch configuration the
benchmark times (default schedule), against the CPU oracle element by element.  The
oracle's column-block OpenMP variant is used so that a case finishes in seconds; it is
pinned to the plain one in test_oracle_pins.py."""
import numpy as np
import pytest

from gpu_util import assert_pad_untouched, assert_parity, require_gpu, same_bits, to_dev
from paper_2507_20424_b200 import inputs

pytestmark = pytest.mark.gpu


def _round_on_gpu(binding, x_np, w, rounds=1):
    import torch
    x = to_dev(x_np)
    norms = torch.zeros(w.M, device="cuda")
    ws = binding.alloc_workspace(w.M, w.d)
    for _ in range(rounds):
        binding.dppf_consensus(x, w.alpha, w.lam, norms_out=norms, ws=ws, d=w.d)
    assert binding.dppf_device_status(ws) == binding.OK
    out, r = x.cpu().numpy(), norms.cpu().numpy()
    del x
    torch.cuda.empty_cache()
    return out, r


@pytest.mark.parametrize("name", ["C1", "C2", "C5"])
def test_single_round_workloads(oracle, name):
    _, binding = require_gpu()
    w = inputs.WORKLOADS[name]
    x = inputs.replicas(w)
    ref, r_ref, _ = oracle.consensus_blocked(x, w.alpha, w.lam, d=w.d)
    got, r = _round_on_gpu(binding, x, w)
    assert_parity(got, r, ref, r_ref, w.d)
    assert_pad_untouched(got, w.d)
    again, r_again = _round_on_gpu(binding, x, w)            # run-to-run reproducible, bit for bit
    assert same_bits(got[:, :w.d], again[:, :w.d]) and same_bits(r, r_again)
    if name == "C1":       # magnitudes the recipe implies: r_m ~ sigma sqrt(d (M-1)/M)
        np.testing.assert_allclose(r, w.drift_std * np.sqrt(w.d * (w.M - 1) / w.M), rtol=0.01)


def test_c5_identical_replicas_round_is_bit_exact(oracle):
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C5"]
    x = inputs.replicas(w, identical=True)
    got, r = _round_on_gpu(binding, x, w)
    assert np.all(r == 0.0)
    assert same_bits(got[:, :w.d], x[:, :w.d])
    assert_pad_untouched(got, w.d)


def test_c4_first_and_hundredth_round(oracle):
    """100 rounds back to back on the device; the oracle iterates 100 times too."""
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C4"]
    x = inputs.replicas(w)
    ref, r_ref, _ = oracle.consensus_blocked(x, w.alpha, w.lam, d=w.d)
    got, r = _round_on_gpu(binding, x, w, rounds=1)
    assert_parity(got, r, ref, r_ref, w.d)
    np.testing.assert_allclose(r, w.drift_std * np.sqrt(w.d * (w.M - 1) / w.M), rtol=0.01)   # 8.058
    for _ in range(w.rounds - 1):
        ref, r_ref, _ = oracle.consensus_blocked(ref, w.alpha, w.lam, d=w.d)
    got, r = _round_on_gpu(binding, x, w, rounds=w.rounds)
    assert_parity(got, r, ref, r_ref, w.d)      # r holds the distances before round 100
    assert_pad_untouched(got, w.d)
    # the valley width has contracted toward lambda/alpha (Theorem 1): r_100 - 0.05 = 0.9^99 (r_1 - 0.05)
    a, l = float(np.float32(w.alpha)), float(np.float32(w.lam))
    assert np.all(np.abs(r_ref - l / a) < 1e-3)


def test_c3_eight_local_steps_then_fused_round(oracle):
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C3"]
    x_np, v_np = inputs.replicas(w), inputs.zeros_like_rows(w)
    x, v = to_dev(x_np), to_dev(v_np)
    x64 = np.array(x_np[:, :w.d], dtype=np.float64)
    v64 = np.zeros_like(x64)
    ws = binding.alloc_workspace(w.M, w.d)
    norms = torch.zeros(w.M, device="cuda")
    for t in range(w.tau):
        g_np = inputs.gradients(w, t)
        x64, v64 = oracle.local_steps_f64(x64, v64, [g_np[:, :w.d]], w.lr, w.momentum, w.weight_decay)
        g = to_dev(g_np)
        if t < w.tau - 1:
            binding.dppf_local_step(x, v, g, w.lr, w.momentum, w.weight_decay, d=w.d)
        else:
            binding.dppf_local_step_and_consensus(x, v, g, w.lr, w.momentum, w.weight_decay,
                                                  w.alpha, w.lam, norms_out=norms, ws=ws, d=w.d)
        torch.cuda.synchronize()
        del g, g_np
    ref, r_ref = oracle.consensus_f64(x64, w.alpha, w.lam)
    assert binding.dppf_device_status(ws) == binding.OK
    got_x, got_v = x.cpu().numpy(), v.cpu().numpy()
    assert_parity(got_x, norms.cpu().numpy(), ref, r_ref, w.d)
    verr = np.abs(got_v[:, :w.d].astype(np.float64) - v64)
    assert np.all(verr <= 1e-6 * (1 + np.abs(v64)))
    assert_pad_untouched(got_x, w.d), assert_pad_untouched(got_v, w.d)
    # per-element displacement std 0.011053 => r ~ 48.4 (shared start, independent gradients)
    np.testing.assert_allclose(r_ref, 48.4, rtol=0.02)


@pytest.mark.parametrize("path", [3, 2])
def test_rows_longer_than_2_to_31_columns(oracle, path):
    """64-bit indexing: d = 2^31 + 4099 columns per row (M = 2, 17 GB on the device).  The
    replicas repeat a random block of P = 2^20 columns, so the CPU oracle can produce the
    exact answer from one period: sum of squares = (d // P) S_P + S_rest, and the update of a
    column depends on the other columns only through r_m, which is matched on a slice by
    rescaling lambda (alpha - lambda'/r_slice = alpha - lambda/r_full)."""
    import torch
    _, binding = require_gpu()
    M, P, d = 2, 1 << 20, (1 << 31) + 4099
    alpha, lam = 0.1, 0.5
    rng = np.random.default_rng(41)
    block = (rng.standard_normal(P)[None, :] * 0.02 + rng.standard_normal((M, P)) * 1e-3).astype(np.float32)
    reps, rest = divmod(d, P)
    x = binding.alloc_rows(M, d)
    blk = torch.from_numpy(block).cuda()
    x[:, :reps * P].view(M, reps, P).copy_(blk[:, None, :].expand(M, reps, P))
    x[:, reps * P:d].copy_(blk[:, :rest])
    x[:, d:].fill_(float("nan"))
    _, r_p = oracle.consensus(block, alpha, 0.0)
    _, r_rest = oracle.consensus(np.ascontiguousarray(block[:, :rest]), alpha, 0.0)
    r_full = np.sqrt(reps * r_p ** 2 + r_rest ** 2)
    norms = torch.zeros(M, device="cuda")
    ws = binding.alloc_workspace(M, d)
    binding.dppf_consensus(x, alpha, lam, norms_out=norms, ws=ws, d=d, path=path)
    assert binding.dppf_device_status(ws) == binding.OK
    r = norms.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(r - r_full) <= 1e-5 * r_full)
    lam32 = float(np.float32(lam))
    # the first period, one in the middle, the last whole one (ends at column 2^31) and the
    # ragged rest beyond 2^31; all of row 1 lies beyond element offset 2^31 as well
    for start, width, r_slice in ((0, P, r_p), (1000 * P, P, r_p), ((reps - 1) * P, P, r_p),
                                  (reps * P, rest, r_rest)):
        ref, _ = oracle.consensus(np.ascontiguousarray(block[:, :width]), alpha, lam32 * r_slice[0] / r_full[0])
        got = x[:, start:start + width].cpu().numpy()
        err = np.abs(got.astype(np.float64) - ref)
        assert np.all(err <= 1e-6 * (1 + np.abs(ref))), (start, float(err.max()))
    assert torch.isnan(x[:, d:]).all()
    del x, blk
    torch.cuda.empty_cache()
