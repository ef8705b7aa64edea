"""Seeded synthetic workloads: shapes, determinism, padding and the magnitudes the
recipes imply (drift N(0, s^2) around a shared point gives r_m ~ s*sqrt(d(M-1)/M))."""
import numpy as np
import pytest

from paper_2507_20424_b200 import inputs


def test_row_stride_is_128_byte_multiple():
    for d, ld in ((1, 32), (32, 32), (33, 64), (25_557_032, 25_557_056), (86_567_656, 86_567_680),
                  (44_549_160, 44_549_184), (26_200_000, 26_200_000), (1 << 20, 1 << 20)):
        assert inputs.row_stride(d) == ld


def test_workload_table_matches_the_five_configs():
    W = inputs.WORKLOADS
    assert [(w.M, w.d) for w in W.values()] == [(4, 1_048_576), (8, 26_200_000), (4, 25_557_032),
                                                (4, 86_567_656), (16, 44_549_160)]
    assert (W["C1"].alpha, W["C1"].lam) == (0.1, 0.01)
    assert (W["C2"].alpha, W["C2"].lam) == (0.05, 0.02)
    assert (W["C3"].tau, W["C3"].lr, W["C3"].momentum, W["C3"].weight_decay) == (8, 0.1, 0.9, 1e-4)
    assert (W["C4"].alpha, W["C4"].lam, W["C4"].rounds) == (0.1, 0.005, 100)
    assert (W["C5"].alpha, W["C5"].lam, W["C5"].drift_log10_range) == (0.2, 0.05, (-5.0, -2.0))


def test_replicas_are_seeded_padded_and_thread_independent():
    w = inputs.WORKLOADS["C1"].scaled(100_003)
    a = inputs.replicas(w, seed=7, threads=1)
    b = inputs.replicas(w, seed=7, threads=4)
    c = inputs.replicas(w, seed=8)
    assert a.shape == (4, 100_032) and a.dtype == np.float32
    assert np.array_equal(a[:, :w.d], b[:, :w.d]) and not np.array_equal(a[:, :w.d], c[:, :w.d])
    assert np.all(np.isnan(a[:, w.d:])) and np.all(np.isfinite(a[:, :w.d]))


def test_magnitudes_c1(oracle):
    w = inputs.WORKLOADS["C1"]
    x = inputs.replicas(w)
    assert abs(x[:, :w.d].std() / w.x0_std - 1) < 0.01
    _, r = oracle.consensus(x, w.alpha, w.lam, d=w.d)
    np.testing.assert_allclose(r, w.drift_std * np.sqrt(w.d * (w.M - 1) / w.M), rtol=0.01)   # 0.887


def test_mixed_scale_drift_and_identical_round():
    w = inputs.WORKLOADS["C5"].scaled(50_000)
    s = inputs.drift_scales(w)
    assert s.shape == (16,) and s.min() >= 1e-5 and s.max() <= 1e-2 and s.max() / s.min() > 30
    x = inputs.replicas(w)
    x0 = inputs.replicas(w, identical=True)
    assert all(np.array_equal(x0[0, :w.d], x0[m, :w.d]) for m in range(16))
    got = (x[:, :w.d] - x0[:, :w.d]).astype(np.float64).std(axis=1)
    np.testing.assert_allclose(got, s, rtol=0.05)


def test_local_step_workload_starts_from_one_shared_point():
    w = inputs.WORKLOADS["C3"].scaled(10_000)
    x = inputs.replicas(w)
    assert all(np.array_equal(x[0, :w.d], x[m, :w.d]) for m in range(w.M))
    v = inputs.zeros_like_rows(w)
    assert np.all(v[:, :w.d] == 0) and np.all(np.isnan(v[:, w.d:]))
    g0, g1 = inputs.gradients(w, 0), inputs.gradients(w, 1)
    assert abs(g0[:, :w.d].std() / w.grad_std - 1) < 0.02
    assert not np.array_equal(g0[:, :w.d], g1[:, :w.d]) and not np.array_equal(g0[0, :w.d], g0[1, :w.d])
    assert np.array_equal(g0[:, :w.d], inputs.gradients(w, 0)[:, :w.d])
