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
    assert binding.dppf_device_schedule(ws) == binding.PATH_STAGED      # bit-for-bit repeats need the same schedule
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


@pytest.fixture(scope="module")
def c4_oracle_rounds(oracle):
    """The oracle's round applied 100 times to the ViT-B/16-sized workload (about 45 s of CPU
    work, shared by the tests below): the input, the state after round 1, the final state and
    the distances before every round."""
    w = inputs.WORKLOADS["C4"]
    x = inputs.replicas(w)
    ref, first, rs = x, None, []
    for k in range(w.rounds):
        ref, r_ref, _ = oracle.consensus_blocked(ref, w.alpha, w.lam, d=w.d)
        rs.append(r_ref)
        if k == 0:
            first = ref
    return x, first, ref, np.array(rs)


def test_c4_first_and_hundredth_round(c4_oracle_rounds):
    """100 rounds back to back on the device, one call per round; the oracle iterates 100 times too."""
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C4"]
    x, first, last, rs = c4_oracle_rounds
    got, r = _round_on_gpu(binding, x, w, rounds=1)
    assert_parity(got, r, first, rs[0], w.d)
    np.testing.assert_allclose(r, w.drift_std * np.sqrt(w.d * (w.M - 1) / w.M), rtol=0.01)   # 8.058
    got, r = _round_on_gpu(binding, x, w, rounds=w.rounds)
    assert_parity(got, r, last, rs[-1], w.d)      # r holds the distances before round 100
    assert_pad_untouched(got, w.d)
    # the valley width has contracted toward lambda/alpha (Theorem 1): r_100 - 0.05 = 0.9^99 (r_1 - 0.05)
    a, l = float(np.float32(w.alpha)), float(np.float32(w.lam))
    assert np.all(np.abs(rs[-1] - l / a) < 1e-3)


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


# ---------------------------------------------------------------- several rounds per launch

def test_c4_hundred_rounds_in_one_call(c4_oracle_rounds):
    """The 100 back-to-back rounds of the ViT-B/16-sized workload as ONE dppf_consensus_rounds call
    (what the benchmark's multi_round figure times): the replicas after round 100 and the
    distances before every one of the 100 rounds against the oracle iterated 100 times."""
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS["C4"]
    x_np, _, ref, rs = c4_oracle_rounds
    outs = []
    for _ in range(2):
        x = to_dev(x_np)
        norms = torch.full((w.rounds, w.M), -1.0, device="cuda")
        ws = binding.alloc_workspace(w.M, w.d)
        binding.dppf_consensus_rounds(x, w.alpha, w.lam, w.rounds, norms_out=norms, ws=ws, d=w.d)
        assert binding.dppf_device_status(ws) == binding.OK
        outs.append((x.cpu().numpy(), norms.cpu().numpy()))
        del x
        torch.cuda.empty_cache()
    got, norms = outs[0]
    assert_parity(got, norms[-1], ref, rs[-1], w.d)
    assert np.all(np.abs(norms - rs) <= 1e-5 * rs)
    assert_pad_untouched(got, w.d)
    assert same_bits(got[:, :w.d], outs[1][0][:, :w.d]) and same_bits(norms, outs[1][1])      # run to run
    np.testing.assert_allclose(norms[0], w.drift_std * np.sqrt(w.d * (w.M - 1) / w.M), rtol=0.01)


@pytest.mark.parametrize("name,n", [("C1", 100), ("C2", 5), ("C5", 3)])
def test_rounds_in_one_call_other_workloads(oracle, name, n):
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS[name]
    x_np = inputs.replicas(w)
    ref, rs = x_np, []
    for _ in range(n):
        ref, r_ref, _ = oracle.consensus_blocked(ref, w.alpha, w.lam, d=w.d)
        rs.append(r_ref)
    rs = np.array(rs)
    x = to_dev(x_np)
    norms = torch.full((n, w.M), -1.0, device="cuda")
    ws = binding.alloc_workspace(w.M, w.d)
    binding.dppf_consensus_rounds(x, w.alpha, w.lam, n, norms_out=norms, ws=ws, d=w.d)
    assert binding.dppf_device_status(ws) == binding.OK
    got, norms = x.cpu().numpy(), norms.cpu().numpy()
    del x
    torch.cuda.empty_cache()
    assert_parity(got, norms[-1], ref, rs[-1], w.d)
    assert np.all(np.abs(norms - rs) <= 1e-5 * rs)
    assert_pad_untouched(got, w.d)


# ---------------------------------------------------------------- general round and AdamW at full size

@pytest.mark.parametrize("name,wkind,push_from,two_term", [("C4", "random", "consensus", True),
                                                           ("C2", "leader", "consensus", False),
                                                           ("C5", "random", "average", True)])
def test_general_round_full_size(oracle, name, wkind, push_from, two_term):
    """Weighted consensus variable / a leader, push from x_A or x_C, one or both gradient terms,
    at the workloads' full sizes (every block wraps its ring many times)."""
    import torch
    _, binding = require_gpu()
    w = inputs.WORKLOADS[name]
    x_np = inputs.replicas(w)
    if wkind == "leader":
        wts = np.zeros(w.M)
        wts[w.M // 2] = 1.0
    else:
        wts = np.random.default_rng(7).random(w.M) + 0.05
    ref, r_ref, n_ref = oracle.consensus_general(x_np, w.alpha, w.lam, wts, push_from, two_term, d=w.d)
    x = to_dev(x_np)
    r = torch.full((w.M,), -1.0, device="cuda")
    n = torch.full((w.M,), -1.0, device="cuda")
    ws = binding.alloc_workspace(w.M, w.d)
    binding.dppf_consensus_general(x, w.alpha, w.lam, wts, {"average": 0, "consensus": 1}[push_from], two_term,
                                   norms_out=r, push_norms_out=n, ws=ws, d=w.d)
    assert binding.dppf_device_status(ws) == binding.OK
    got = x.cpu().numpy()
    del x
    torch.cuda.empty_cache()
    assert_parity(got, r.cpu().numpy(), ref, r_ref, w.d)
    assert np.all(np.abs(n.cpu().numpy() - n_ref) <= 1e-5 * n_ref)
    assert_pad_untouched(got, w.d)


def test_adamw_steps_then_fused_round_at_vit_size(oracle):
    """The paper's ViT setting (AdamW, lr 5e-4, weight decay 0.01) at the ViT-B/16-sized
    workload: one stand-alone AdamW step, then the second step fused with the round; replicas,
    both moment buffers and the distances against the fp64 oracle."""
    import torch
    from dataclasses import replace
    _, binding = require_gpu()
    hp = dict(lr=5e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    w = replace(inputs.WORKLOADS["C4"], grad_std=1e-2, alpha=0.9, lam=0.09)
    x_np = inputs.replicas(w)
    x = to_dev(x_np)
    a, b = binding.alloc_rows(w.M, w.d, fill=0.0), binding.alloc_rows(w.M, w.d, fill=0.0)
    x64 = np.array(x_np[:, :w.d], dtype=np.float64)
    a64, b64 = np.zeros_like(x64), np.zeros_like(x64)
    norms = torch.zeros(w.M, device="cuda")
    ws = binding.alloc_workspace(w.M, w.d)
    for t in range(2):
        g_np = inputs.gradients(w, t)
        x64, a64, b64 = oracle.adamw_steps_f64(x64, a64, b64, [g_np[:, :w.d]], first_step=t + 1, **hp)
        g = to_dev(g_np)
        if t == 0:
            binding.dppf_adamw_step(x, a, b, g, step=1, d=w.d, **hp)
        else:
            binding.dppf_adamw_step_and_consensus(x, a, b, g, step=2, alpha=w.alpha, lam=w.lam, norms_out=norms,
                                                  ws=ws, d=w.d, **hp)
        torch.cuda.synchronize()
        del g, g_np
    ref, r_ref = oracle.consensus_f64(x64, w.alpha, w.lam)
    del x64
    assert binding.dppf_device_status(ws) == binding.OK
    got_x = x.cpu().numpy()
    assert_parity(got_x, norms.cpu().numpy(), ref, r_ref, w.d)
    assert_pad_untouched(got_x, w.d)
    for got, want in ((a.cpu().numpy()[:, :w.d], a64), (b.cpu().numpy()[:, :w.d], b64)):
        err = np.abs(got.astype(np.float64) - want)
        assert np.all(err <= 2e-6 * np.abs(want).max() + 1e-5 * np.abs(want))
    del x, a, b
    torch.cuda.empty_cache()
