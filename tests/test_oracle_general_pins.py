"""Pins for the general-round oracle (arbitrary consensus variable, push from x_A or x_C,
optional second gradient term): hand cases, a finite-difference check against the
regulariser R = -(1/M) sum ||x_i - x_A|| itself, conservation laws and special cases."""
import json
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def replicas(seed, M, d, base=0.5, drift=0.2):
    rng = np.random.default_rng(seed)
    return f32(rng.standard_normal(d)[None, :] * base + rng.standard_normal((M, d)) * drift)


def test_hand_cases(oracle):
    with open(os.path.join(GOLD, "general_round_cases.json")) as f:
        g = json.load(f)
    for c in g["cases"]:
        xp, r, n = oracle.consensus_general(f32(g["x"]), g["alpha"], g["lambda"], g["weights"],
                                            c["push_from"], c["two_term"])
        assert np.array_equal(xp, f32(c["x_plus"])), c["name"]
        assert np.array_equal(r, c["r"]) and np.array_equal(n, c["n"]), c["name"]


@pytest.mark.parametrize("alpha,lam", [(0.1, 0.01), (0.5, 5.0), (0.9, 0.3), (0.05, 0.0)])
def test_default_arguments_reduce_to_the_single_line_update(oracle, alpha, lam):
    x = replicas(1, 5, 301)
    a, r = oracle.consensus(x, alpha, lam)
    for w in (None, np.full(5, 1.0), np.full(5, 0.2)):
        b, r2, n = oracle.consensus_general(x, alpha, lam, w)
        np.testing.assert_allclose(r2, r, rtol=1e-15)
        np.testing.assert_allclose(n, (1 - float(np.float32(alpha))) * r, rtol=1e-12)
        assert np.max(np.abs(a.astype(np.float64) - b)) <= 2.4e-7


def test_two_term_push_is_minus_lambda_M_times_the_gradient_of_R(oracle):
    """alpha = 0: x+ - x = lambda (u_m - ubar) = -lambda M dR/dx_m, R differentiated numerically."""
    M, d, lam = 3, 4, 0.25
    x = replicas(2, M, d)

    def R(z):
        zA = z.mean(axis=0)
        return -np.mean(np.linalg.norm(z - zA, axis=1))

    x64 = x.astype(np.float64)
    grad = np.zeros_like(x64)
    h = 1e-6
    for m in range(M):
        for i in range(d):
            zp, zm = x64.copy(), x64.copy()
            zp[m, i] += h
            zm[m, i] -= h
            grad[m, i] = (R(zp) - R(zm)) / (2 * h)
    xp, _, _ = oracle.consensus_general(x, 0.0, lam, None, "average", True)
    np.testing.assert_allclose(xp.astype(np.float64) - x64, -lam * M * grad, rtol=0, atol=2e-7)
    # the one-term push keeps only the first part: M * (lambda / M) u_m
    xq, r, _ = oracle.consensus_general(x, 0.0, lam, None, "average", False)
    u = (x64 - x64.mean(axis=0)) / r[:, None]
    np.testing.assert_allclose(xq.astype(np.float64) - x64, lam * u, rtol=0, atol=1e-7)


@pytest.mark.parametrize("push_from", ["average", "consensus"])
def test_two_term_push_conserves_the_mean_of_the_pulled_points(oracle, push_from):
    M, d, alpha, lam = 6, 400, 0.3, 0.7
    x = replicas(3, M, d)
    w = np.random.default_rng(3).random(M) + 0.1
    xp, _, _ = oracle.consensus_general(x, alpha, lam, w, push_from, True)
    a = float(np.float32(alpha))
    w32 = w.astype(np.float32).astype(np.float64)
    xA, xC = x.astype(np.float64).mean(axis=0), (w32[:, None] * x).sum(axis=0) / w32.sum()
    np.testing.assert_allclose(xp.astype(np.float64).mean(axis=0), (1 - a) * xA + a * xC, rtol=0, atol=1e-7)
    # without the second term the mean moves by lambda * ubar
    xq, _, n = oracle.consensus_general(x, alpha, lam, w, push_from, False)
    y = (1 - a) * x.astype(np.float64) + a * xC
    P = xA if push_from == "average" else xC
    ubar = ((y - P) / n[:, None]).mean(axis=0)
    np.testing.assert_allclose(xq.astype(np.float64).mean(axis=0), (1 - a) * xA + a * xC + float(np.float32(lam)) * ubar,
                               rtol=0, atol=1e-7)
    np.testing.assert_allclose(np.linalg.norm(xq - y, axis=1), float(np.float32(lam)), rtol=1e-6)


def test_leader_as_consensus_variable(oracle):
    """One-hot weights: every worker is pulled toward the leader; pushing from the leader
    leaves the leader where it is and moves the others straight away from it."""
    M, d, L = 4, 257, 2
    x = replicas(4, M, d)
    w = np.zeros(M)
    w[L] = 1.0
    xp, r, n = oracle.consensus_general(x, 0.25, 0.125, w, "consensus", False)
    assert np.array_equal(xp[L], x[L]) and n[L] == 0.0
    y = 0.75 * x.astype(np.float64) + 0.25 * x[L].astype(np.float64)
    for m in range(M):
        if m == L:
            continue
        step = xp[m].astype(np.float64) - y[m]
        np.testing.assert_allclose(np.linalg.norm(step), 0.125, rtol=1e-5)
        away = y[m] - x[L]
        assert np.dot(step, away) / (np.linalg.norm(step) * np.linalg.norm(away)) > 1 - 1e-6
        np.testing.assert_allclose(n[m], 0.75 * np.linalg.norm(x[m].astype(np.float64) - x[L]), rtol=1e-12)
    # pushing from the average instead is not aligned with the pull toward the leader
    xq, _, _ = oracle.consensus_general(x, 0.25, 0.125, w, "average", False)
    assert not np.allclose(xq, xp)


def test_weights_are_normalised_and_pad_columns_ignored(oracle):
    x = np.full((3, 64), np.nan, dtype=np.float32)
    x[:, :41] = replicas(5, 3, 41)
    w = np.array([0.5, 0.25, 1.0])
    a, r, n = oracle.consensus_general(x, 0.2, 0.3, w, "consensus", True, d=41)
    b, r2, n2 = oracle.consensus_general(x, 0.2, 0.3, 4.0 * w, "consensus", True, d=41)
    assert np.array_equal(a[:, :41], b[:, :41]) and np.all(np.isnan(a[:, 41:])) and np.all(np.isfinite(a[:, :41]))
    np.testing.assert_allclose(r, r2, rtol=0) and np.testing.assert_allclose(n, n2, rtol=0)


@pytest.mark.parametrize("M", [1, 2, 5])
def test_identical_replicas_are_copied_unchanged(oracle, M):
    row = replicas(6, 1, 300)
    row[0, [1, 17]] = np.float32(-0.0)
    x = np.repeat(row, M, axis=0)
    for two in (False, True):
        xp, r, n = oracle.consensus_general(x, 0.2, 0.05, np.arange(1, M + 1), "consensus", two)
        assert np.array_equal(xp.view(np.uint32), x.view(np.uint32)) and np.all(r == 0) and np.all(n == 0)
