"""Pins for the CPU oracle: hand cases, closed forms, identities from the proof of
Theorem 1, exact-arithmetic brute force and library special cases.  None of these
re-type the oracle's own formula; each checks a property that the single-line
update (Sec. 5) must have, or a value worked out by other means."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
from mpmath import mp, mpf, sqrt as mpsqrt

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def rand_replicas(rng, M, d, base=0.02, drift=1e-3):
    x0 = rng.standard_normal(d) * base
    return f32(x0[None, :] + rng.standard_normal((M, d)) * drift)


def mean64(x):
    return np.asarray(x, dtype=np.float64).mean(axis=0)


# ---------------------------------------------------------------- hand cases

def _hand_cases():
    with open(os.path.join(GOLD, "hand_cases.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _hand_cases(), ids=lambda c: c["name"].split(":")[0])
@pytest.mark.parametrize("fn", ["consensus", "consensus_two_step", "consensus_blocked"])
def test_hand_cases(oracle, case, fn):
    if fn == "consensus_two_step" and case["alpha"] >= 1.0:
        pytest.skip("two-step form is 0/0 at alpha = 1")
    out = getattr(oracle, fn)(f32(case["x"]), case["alpha"], case["lambda"])
    xp, r = out[0], out[1]
    tol = case["tol"]
    np.testing.assert_allclose(r, case["r"], rtol=1e-15, atol=0)
    if tol == 0.0:
        assert np.array_equal(xp, f32(case["x_plus"]))
    else:
        np.testing.assert_allclose(xp, case["x_plus"], rtol=0, atol=tol)


# ------------------------------------------------- exact brute force, tiny inputs

def _exact_round(x, alpha32, lam32):
    """Algorithm 1's two lines (pull, then push) in exact rational arithmetic, the
    only irrational step (the norm) taken to 60 digits.  The squared norm uses the
    expansion |x|^2 - 2 x.A + |A|^2 rather than a sum of squared differences."""
    mp.dps = 60
    M, d = x.shape
    X = [[Fraction(float(v)) for v in row] for row in x]
    a, lam = Fraction(float(np.float32(alpha32))), Fraction(float(np.float32(lam32)))
    A = [sum(X[m][i] for m in range(M)) / M for i in range(d)]
    AA = sum(v * v for v in A)
    outs, rs = [], []
    for m in range(M):
        S = sum(v * v for v in X[m]) - 2 * sum(X[m][i] * A[i] for i in range(d)) + AA
        rs.append(mpsqrt(mpf(S.numerator) / mpf(S.denominator)))
        y = [(1 - a) * X[m][i] + a * A[i] for i in range(d)]            # pull
        S1 = sum((y[i] - A[i]) ** 2 for i in range(d))
        n1 = mpsqrt(mpf(S1.numerator) / mpf(S1.denominator))
        row = []
        for i in range(d):
            yi = mpf(y[i].numerator) / mpf(y[i].denominator)
            di = y[i] - A[i]
            push = mpf(lam.numerator) / mpf(lam.denominator) * (mpf(di.numerator) / mpf(di.denominator)) / n1 if n1 > 0 else mpf(0)
            row.append(yi + push)                                        # push
        outs.append(row)
    return outs, rs


@pytest.mark.parametrize("M,d,alpha,lam", [(2, 1, 0.1, 0.5), (2, 3, 0.3, 0.05), (3, 5, 0.1, 0.01),
                                            (4, 7, 0.05, 0.02), (5, 4, 0.9, 9.0), (16, 3, 0.2, 0.05)])
def test_exact_brute_force(oracle, M, d, alpha, lam):
    rng = np.random.default_rng(1000 * M + d)
    x = rand_replicas(rng, M, d, base=0.5, drift=0.2)
    xp, r = oracle.consensus(x, alpha, lam)
    ex, er = _exact_round(x, alpha, lam)
    for m in range(M):
        assert abs(mpf(float(r[m])) - er[m]) <= abs(er[m]) * mpf(4e-16)
        for i in range(d):
            exact = ex[m][i]
            ulp = float(np.spacing(np.float32(abs(float(exact)))))
            assert abs(mpf(float(xp[m, i])) - exact) <= 0.5000001 * ulp, (m, i)


# ------------------------------------------------------- invariants of the update

def test_alpha_one_lambda_zero_collapses_onto_average(oracle):
    # LocalSGD hard reset (Sec. 3): alpha = 1, no push  =>  every replica becomes x_A
    x = rand_replicas(np.random.default_rng(1), 5, 257)
    xp, _ = oracle.consensus(x, 1.0, 0.0)
    A = mean64(x)
    for m in range(5):
        assert np.array_equal(xp[m], A.astype(np.float32))


def test_lambda_zero_preserves_average(oracle):
    x = rand_replicas(np.random.default_rng(2), 6, 1001)
    for alpha in (0.05, 0.1, 0.5, 0.9):
        xp, _ = oracle.consensus(x, alpha, 0.0)
        np.testing.assert_allclose(mean64(xp), mean64(x), rtol=0, atol=3e-9)


def test_alpha_zero_displacement_has_norm_lambda(oracle):
    # the push is unit-normed and scaled by lambda (Sec. 5, after the regulariser gradient)
    x = rand_replicas(np.random.default_rng(3), 4, 4097, base=1.0, drift=0.5)
    for lam in (0.03, 0.5, 9.0):
        xp, _ = oracle.consensus(x, 0.0, lam)
        disp = np.linalg.norm(xp.astype(np.float64) - x.astype(np.float64), axis=1)
        np.testing.assert_allclose(disp, float(np.float32(lam)), rtol=2e-6)
        # and it points away from the average
        A = mean64(x)
        assert np.all(np.einsum("md,md->m", xp.astype(np.float64) - x, x - A) > 0)


def test_single_worker_unchanged(oracle):
    x = rand_replicas(np.random.default_rng(4), 1, 300)
    xp, r = oracle.consensus(x, 0.3, 0.7)
    assert np.array_equal(xp, x) and r[0] == 0.0


@pytest.mark.parametrize("M", [2, 3, 4, 7, 16])
def test_identical_replicas_unchanged_bit_exact(oracle, M):
    row = rand_replicas(np.random.default_rng(5), 1, 777)
    row[0, [3, 500]] = np.float32(-0.0)          # "unchanged" includes the sign of a zero
    row[0, 7] = np.float32(0.0)
    x = np.repeat(row, M, axis=0)
    for fn in (oracle.consensus, oracle.consensus_two_step, lambda *a: oracle.consensus_blocked(*a)[:2]):
        xp, r = fn(x, 0.2, 0.05)
        assert np.array_equal(xp.view(np.uint32), x.view(np.uint32))
        assert np.all(r == 0.0)


def test_two_workers_keep_average_and_follow_scalar_recurrence(oracle):
    # M = 2: u_1 = -u_2, so the sum of unit directions vanishes and the gap obeys
    # r+ = |(1 - alpha) r + lambda| exactly (gap recurrence in the proof of Theorem 1)
    x = rand_replicas(np.random.default_rng(6), 2, 513, base=1.0, drift=0.3)
    for alpha, lam in ((0.1, 0.5), (0.5, 5.0), (0.9, 0.03)):
        xp, r = oracle.consensus(x, alpha, lam)
        np.testing.assert_allclose(mean64(xp), mean64(x), rtol=0, atol=2e-7)
        _, rp = oracle.consensus(xp, alpha, lam)
        a, l = float(np.float32(alpha)), float(np.float32(lam))
        np.testing.assert_allclose(rp, np.abs((1 - a) * r + l), rtol=3e-6)


@pytest.mark.parametrize("alpha,lam", [(0.1, 0.01), (0.05, 0.02), (0.2, 0.05), (0.9, 9.0), (0.0, 0.3)])
def test_distance_to_old_average(oracle, alpha, lam):
    # from the update: x+_m - x_A = (x_m - x_A)(1 - alpha + lambda/r_m), same direction
    x = rand_replicas(np.random.default_rng(7), 8, 2049, base=0.05, drift=5e-3)
    xp, r = oracle.consensus(x, alpha, lam)
    A = mean64(x)
    a, l = float(np.float32(alpha)), float(np.float32(lam))
    got = np.linalg.norm(xp.astype(np.float64) - A, axis=1)
    np.testing.assert_allclose(r, np.linalg.norm(x.astype(np.float64) - A, axis=1), rtol=1e-13)
    np.testing.assert_allclose(got, np.abs((1 - a) * r + l), rtol=2e-6)
    cos = np.einsum("md,md->m", xp - A, x - A) / (got * r)
    np.testing.assert_allclose(cos, np.sign((1 - a) * r + l), atol=1e-9)


def test_gap_identity_and_new_average_from_proof(oracle):
    # Theorem 1 proof: with Delta = x_A - x_m, u = Delta/|Delta|:
    #   x_A+    = x_A - (lambda/M) sum_i u_i
    #   Delta_m+ = (1 - alpha) Delta_m + lambda u_m - (lambda/M) sum_i u_i
    M, d = 5, 1500
    x = rand_replicas(np.random.default_rng(8), M, d, base=0.3, drift=0.1)
    alpha, lam = 0.3, 0.25
    xp, r = oracle.consensus(x, alpha, lam)
    a, l = float(np.float32(alpha)), float(np.float32(lam))
    A = mean64(x)
    Delta = A - x.astype(np.float64)
    u = Delta / np.linalg.norm(Delta, axis=1, keepdims=True)
    ubar = u.mean(axis=0)
    np.testing.assert_allclose(mean64(xp), A - l * ubar, rtol=0, atol=1e-7)
    Dp = mean64(xp) - xp.astype(np.float64)
    np.testing.assert_allclose(Dp, (1 - a) * Delta + l * u - l * ubar, rtol=0, atol=1e-7)


def test_symmetries(oracle):
    rng = np.random.default_rng(9)
    M, d = 4, 640
    x = rand_replicas(rng, M, d, base=0.5, drift=0.25)
    alpha, lam = 0.125, 0.5
    xp, r = oracle.consensus(x, alpha, lam)
    pm, pc = rng.permutation(M), rng.permutation(d)
    xq, rq = oracle.consensus(f32(x[pm]), alpha, lam)                 # worker permutation
    np.testing.assert_allclose(xq, xp[pm], rtol=0, atol=1e-7); np.testing.assert_allclose(rq, r[pm], rtol=1e-13)
    xq, rq = oracle.consensus(f32(x[:, pc]), alpha, lam)              # coordinate permutation
    np.testing.assert_allclose(xq, xp[:, pc], rtol=0, atol=1e-7); np.testing.assert_allclose(rq, r, rtol=1e-13)
    xq, rq = oracle.consensus(f32(x + 8.0), alpha, lam)               # translation (8 + x exact enough)
    np.testing.assert_allclose(xq, xp + 8.0, rtol=0, atol=2e-6); np.testing.assert_allclose(rq, r, rtol=1e-5)
    xq, rq = oracle.consensus(f32(4.0 * x), alpha, 4.0 * lam)         # scaling by a power of two is exact
    assert np.array_equal(xq, 4.0 * xp); np.testing.assert_allclose(rq, 4.0 * r, rtol=1e-15)


def test_two_step_form_equals_single_line_for_alpha_below_one(oracle):
    x = rand_replicas(np.random.default_rng(10), 6, 999, base=0.1, drift=0.02)
    for alpha, lam in ((0.05, 0.02), (0.1, 0.5), (0.5, 5.0), (0.9, 9.0)):
        a1, r1 = oracle.consensus(x, alpha, lam)
        a2, r2 = oracle.consensus_two_step(x, alpha, lam)
        np.testing.assert_allclose(r1, r2, rtol=1e-15)
        np.testing.assert_allclose(a1, a2, rtol=0, atol=1e-6 * (1 + np.abs(a1).max()) * 1e-1)


def test_blocked_variant_matches_plain(oracle):
    x = rand_replicas(np.random.default_rng(11), 7, 12345)
    a1, r1 = oracle.consensus(x, 0.1, 0.01)
    for th in (1, 2, 3, 8):
        a2, r2, used = oracle.consensus_blocked(x, 0.1, 0.01, threads=th)
        assert used == th
        np.testing.assert_allclose(r2, r1, rtol=1e-13)
        assert np.max(np.abs(a2.astype(np.float64) - a1)) <= 2e-9


def test_pad_columns_are_never_read_or_written(oracle):
    x = np.full((3, 64), np.nan, dtype=np.float32)
    x[:, :37] = rand_replicas(np.random.default_rng(12), 3, 37)
    for fn in (oracle.consensus, oracle.consensus_two_step):
        xp, r = fn(x, 0.1, 0.01, d=37)
        assert np.all(np.isfinite(r)) and np.all(np.isfinite(xp[:, :37])) and np.all(np.isnan(xp[:, 37:]))
    xp2, r2 = oracle.consensus(np.ascontiguousarray(x[:, :37]), 0.1, 0.01)
    assert np.array_equal(xp[:, :37], xp2)


# ------------------------------------------------ iteration: valley width lambda/alpha

def _simplex(M, d, radius, rng):
    """M points at the vertices of a regular simplex centred at a random point
    (sum of unit directions = 0, the symmetric arrangement of the appendix)."""
    E = np.eye(M) - 1.0 / M
    E /= np.linalg.norm(E, axis=1, keepdims=True)
    Q, _ = np.linalg.qr(rng.standard_normal((d, M)))
    return f32(rng.standard_normal(d)[None, :] + radius * (E @ Q.T))


@pytest.mark.parametrize("M", [2, 4, 8])
def test_noise_free_iteration_settles_at_lambda_over_alpha(oracle, M):
    with open(os.path.join(GOLD, "paper_values.json")) as f:
        g = json.load(f)["steady_state_distance"]
    alpha, lam = g["alpha"], g["lambda"]
    a, l = float(np.float32(alpha)), float(np.float32(lam))
    x = _simplex(M, 64, 1.0, np.random.default_rng(13))
    r0 = None
    for k in range(200):
        xn, r = oracle.consensus(x, alpha, lam)
        if r0 is None:
            r0 = r.copy()
        # r_k = lambda/alpha + (1 - alpha)^k (r_0 - lambda/alpha)   (geometric recursion, Theorem 1 proof)
        np.testing.assert_allclose(r, l / a + (1 - a) ** k * (r0 - l / a), rtol=2e-5)
        x = xn
    np.testing.assert_allclose(r, g["value"], rtol=1e-4)


def test_mean_direction_norm_is_about_one_over_sqrt_M(oracle):
    # Lemma 2: E|ubar|^2 = 1/M for independent directions; the new average moves by lambda*|ubar|
    M, d, lam = 8, 20000, 0.5
    x = rand_replicas(np.random.default_rng(14), M, d)
    xp, _ = oracle.consensus(x, 0.1, lam)
    shift = np.linalg.norm(mean64(xp) - mean64(x)) / lam
    # drift directions about a sample mean are negatively correlated: |ubar| is well below 1/sqrt(M)
    assert shift < 1.0 / np.sqrt(M)


# ------------------------------------------------------------- local optimiser step

def test_local_step_closed_form_constant_gradient(oracle):
    with open(os.path.join(GOLD, "paper_values.json")) as f:
        g = json.load(f)["momentum_closed_form"]
    tau, mu = g["tau"], g["momentum"]
    M, d, lr = 2, 50, 0.1
    rng = np.random.default_rng(15)
    x0 = rand_replicas(rng, M, d)
    grad = f32(rng.standard_normal((M, d)) * 1e-2)
    x64, v64 = oracle.local_steps_f64(x0, np.zeros_like(x0), [grad] * tau, lr, mu, 0.0)
    mu32, lr32 = float(np.float32(mu)), float(np.float32(lr))
    factor = (tau - mu32 * (1 - mu32 ** tau) / (1 - mu32)) / (1 - mu32)
    assert abs(factor - g["factor"]) < 1e-5
    np.testing.assert_allclose(x64, x0.astype(np.float64) - lr32 * factor * grad.astype(np.float64), rtol=0, atol=1e-15)
    np.testing.assert_allclose(v64, grad.astype(np.float64) * (1 - mu32 ** tau) / (1 - mu32), rtol=1e-13)


def test_local_step_weight_decay_only_is_geometric_shrink(oracle):
    # g = 0, momentum = 0: x <- x (1 - lr wd) each step
    x0 = rand_replicas(np.random.default_rng(16), 3, 40)
    zero = np.zeros_like(x0)
    x64, _ = oracle.local_steps_f64(x0, zero, [zero] * 5, 0.1, 0.0, 0.01)
    k = 1.0 - float(np.float32(0.1)) * float(np.float32(0.01))
    np.testing.assert_allclose(x64, x0.astype(np.float64) * k ** 5, rtol=1e-14)


def test_local_step_matches_library_sgd(oracle):
    # the reading of the optimiser is the documented torch.optim.SGD recurrence
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(17)
    M, d, tau = 3, 101, 8
    lr, mu, wd = 0.1, 0.9, 1e-4
    x0 = rand_replicas(rng, M, d)
    grads = [f32(rng.standard_normal((M, d)) * 1e-2) for _ in range(tau)]
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(mu)),
                          weight_decay=float(np.float32(wd)), dampening=0, nesterov=False)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
    x64, v64 = oracle.local_steps_f64(x0, np.zeros_like(x0), grads, lr, mu, wd)
    np.testing.assert_allclose(x64, p.detach().numpy(), rtol=0, atol=1e-15)
    np.testing.assert_allclose(v64, opt.state[p]["momentum_buffer"].numpy(), rtol=0, atol=1e-15)


def test_local_steps_then_round_composes(oracle):
    rng = np.random.default_rng(18)
    M, d = 4, 333
    x0 = np.repeat(rand_replicas(rng, 1, d), M, axis=0)
    grads = [f32(rng.standard_normal((M, d)) * 1e-2) for _ in range(3)]
    xp, v64, r = oracle.local_steps_then_consensus(x0, np.zeros_like(x0), grads, 0.1, 0.9, 1e-4, 0.1, 0.01)
    x64, _ = oracle.local_steps_f64(x0, np.zeros_like(x0), grads, 0.1, 0.9, 1e-4)
    # same invariant as test_distance_to_old_average, on the stepped state
    A = x64.mean(axis=0)
    a, l = float(np.float32(0.1)), float(np.float32(0.01))
    np.testing.assert_allclose(np.linalg.norm(xp - A, axis=1), np.abs((1 - a) * r + l), rtol=2e-6)
    np.testing.assert_allclose(r, np.linalg.norm(x64 - A, axis=1), rtol=1e-13)


# ------------------------------------------------------------- AdamW local step

def test_adamw_first_step_is_a_signed_step_of_size_lr(oracle):
    # t = 1, zero moments: m/(1-b1) = g, v/(1-b2) = g^2  =>  x1 = x0 (1 - lr wd) - lr g / (|g| + eps)
    rng = np.random.default_rng(21)
    x0 = rand_replicas(rng, 2, 60)
    g = f32(rng.standard_normal((2, 60)) * 1e-2)
    z = np.zeros_like(x0)
    lr, wd, eps = 5e-4, 0.01, 1e-8
    x64, a64, b64 = oracle.adamw_steps_f64(x0, z, z, [g], lr, 0.9, 0.999, eps, wd)
    lr32, wd32, eps32 = (float(np.float32(v)) for v in (lr, wd, eps))
    g64 = g.astype(np.float64)
    np.testing.assert_allclose(x64, x0.astype(np.float64) * (1 - lr32 * wd32) - lr32 * g64 / (np.abs(g64) + eps32),
                               rtol=0, atol=1e-12)
    np.testing.assert_allclose(a64, (1 - float(np.float32(0.9))) * g64, rtol=1e-14)
    np.testing.assert_allclose(b64, (1 - float(np.float32(0.999))) * g64 ** 2, rtol=1e-14)


def test_adamw_matches_library_adamw(oracle):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(22)
    M, d, tau = 3, 77, 6
    lr, b1, b2, eps, wd = 5e-4, 0.9, 0.999, 1e-8, 0.01
    x0 = rand_replicas(rng, M, d)
    grads = [f32(rng.standard_normal((M, d)) * 1e-2) for _ in range(tau)]
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    f = lambda v: float(np.float32(v))
    opt = torch.optim.AdamW([p], lr=f(lr), betas=(f(b1), f(b2)), eps=f(eps), weight_decay=f(wd), amsgrad=False)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
    z = np.zeros_like(x0)
    x64, a64, b64 = oracle.adamw_steps_f64(x0, z, z, grads, lr, b1, b2, eps, wd)
    np.testing.assert_allclose(x64, p.detach().numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(a64, opt.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(b64, opt.state[p]["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-20)
    # continuing from step 4 gives the same state as running straight through
    xa, aa, ba = oracle.adamw_steps_f64(x0, z, z, grads[:3], lr, b1, b2, eps, wd)
    xb, ab, bb = oracle.adamw_steps_f64(xa, aa, ba, grads[3:], lr, b1, b2, eps, wd, first_step=4)
    assert np.array_equal(xb, x64) and np.array_equal(ab, a64) and np.array_equal(bb, b64)


# ---------------------------------------------------------------- one worker given the average

def test_worker_update_hand_cases(oracle):
    """By hand from the single-line update: x = (0, 0), x_A = (3, 4): r = 5.  alpha = 1/8, lambda = 5/8
    (both exact in fp32, lambda / alpha = 5) is the fixed point (c = 0); alpha = 0.5, lambda = 0 moves half
    way; alpha = 0, lambda = 1 moves one
    unit AWAY from x_A along (x - x_A)/r = (-0.6, -0.8)."""
    x, red = np.zeros(2, dtype=np.float32), np.array([6.0, 8.0], dtype=np.float32)
    out, r = oracle.worker_update(x, red, 0.5, 0.125, 0.625)
    assert r == 5.0 and np.array_equal(out, x)
    out, r = oracle.worker_update(x, red, 0.5, 0.5, 0.0)
    assert np.array_equal(out, np.array([1.5, 2.0], dtype=np.float32))
    out, r = oracle.worker_update(x, red, 0.5, 0.0, 1.0)
    np.testing.assert_allclose(out, [-0.6, -0.8], rtol=1e-7)
    out, r = oracle.worker_update(red, red, 1.0, 0.3, 0.7)          # the worker sits on the average
    assert r == 0.0 and np.array_equal(out, red)


def test_worker_update_is_one_row_of_the_round(oracle):
    """Every worker applying its own update with the shared average reproduces the round on
    all replicas (the average handed over as fp32, hence a few fp32 ulps of slack)."""
    rng = np.random.default_rng(11)
    M, d = 5, 4001
    x = (rng.standard_normal(d) * 0.02 + rng.standard_normal((M, d)) * 1e-3).astype(np.float32)
    ref, r_ref = oracle.consensus(x, 0.2, 0.05)
    total = x.astype(np.float64).sum(axis=0).astype(np.float32)
    for m in range(M):
        out, r = oracle.worker_update(x[m], total, 1.0 / M, 0.2, 0.05)
        assert abs(r - r_ref[m]) <= 1e-6 * r_ref[m]
        np.testing.assert_allclose(out, ref[m], rtol=0, atol=2e-8)
