"""Host-side scalars: the library's schedule and metric helpers against the Python oracle,
and the oracle against the values the formulas fix (end points, mid point, complementarity,
the paper's own QSR parameter pairs)."""
import math

import numpy as np
import pytest

from oracle import schedules as ref


@pytest.fixture(scope="module")
def b():
    from paper_2507_20424_b200 import binding, build
    build.build()
    binding.load()
    return binding


def test_oracle_schedule_end_points_and_symmetry():
    lam, T = 0.5, 1000
    assert ref.lambda_schedule(ref.DECREASING, lam, 0, T) == lam
    assert abs(ref.lambda_schedule(ref.DECREASING, lam, T, T)) < 1e-16
    assert ref.lambda_schedule(ref.INCREASING, lam, 0, T) == 0.0
    assert abs(ref.lambda_schedule(ref.INCREASING, lam, T, T) - lam) < 1e-16
    for t in (0, 1, 250, 500, 999, 1000):
        inc, dec = ref.lambda_schedule(ref.INCREASING, lam, t, T), ref.lambda_schedule(ref.DECREASING, lam, t, T)
        assert abs(inc + dec - lam) < 1e-15                       # the two cosine schedules are mirror images
        assert ref.lambda_schedule(ref.FIXED, lam, t, T) == lam
        assert abs(dec - ref.lr_cosine(lam, t, T)) < 1e-16          # "decayed in parallel with the learning rate"
    assert abs(ref.lambda_schedule(ref.INCREASING, lam, 500, T) - lam / 2) < 1e-16
    assert abs(ref.lambda_schedule(ref.INCREASING, lam, 250, T) - lam * (1 - math.sqrt(0.5)) / 2) < 1e-15
    vals = [ref.lambda_schedule(ref.INCREASING, lam, t, T) for t in range(T + 1)]
    assert all(x <= y for x, y in zip(vals, vals[1:]))


def test_oracle_qsr_rule():
    # beta = 0.2, 0.25, 0.3 at eta_max = 0.8 (the cited setting): (beta/eta)^2 < 1 -> tau_base
    for beta in (0.2, 0.25, 0.3):
        assert ref.qsr_period(4, beta, 0.8) == 4
    assert ref.qsr_period(2, 0.2, 0.05) == 16 and ref.qsr_period(2, 0.3, 0.01) == 900
    assert ref.qsr_period(8, 0.2, 0.1) == 8                        # floor(4) = 4 < tau_base
    # the paper rescales beta with eta_max so that beta/eta is unchanged: same periods
    for frac in (1.0, 0.5, 0.1, 0.03):
        a = ref.qsr_period(4, 0.25, 0.8 * frac)
        assert a == ref.qsr_period(4, 0.03125, 0.1 * frac) == ref.qsr_period(4, 0.234375, 0.75 * frac)


def test_oracle_round_metrics():
    mean, pull, push = ref.round_metrics([5.0, 5.0, 5.0, 5.0], 0.1, 0.5)
    assert mean == 5.0 and push == 0.5 and all(abs(p - 0.5) < 1e-15 for p in pull)   # balance at lambda/alpha
    mean, pull, push = ref.round_metrics([1.0, 3.0], 0.5, 0.25)
    assert mean == 2.0 and pull == [0.5, 1.5] and push == 0.25


def test_library_matches_oracle(b):
    f = lambda v: float(np.float32(v))
    for kind in (ref.FIXED, ref.DECREASING, ref.INCREASING):
        for lam in (0.5, 9.0, 0.03):
            for t, T in ((0, 100), (37, 100), (100, 100), (123456, 1000000)):
                got = b.dppf_lambda_schedule(kind, lam, t, T)
                assert abs(got - ref.lambda_schedule(kind, f(lam), t, T)) <= 1e-7 * f(lam)
    assert math.isnan(b.dppf_lambda_schedule(7, 0.5, 1, 10)) and math.isnan(b.dppf_lambda_schedule(1, 0.5, 1, 0))
    assert b.dppf_lambda_schedule(0, 0.5, 1, 0) == 0.5
    for t in (0, 10, 50, 99, 100):
        assert abs(b.dppf_lr_cosine(0.1, t, 100) - ref.lr_cosine(f(0.1), t, 100)) <= 1e-8
    for tau_base, beta, lr in ((4, 0.2, 0.8), (2, 0.2, 0.05), (2, 0.3, 0.01), (8, 0.2, 0.1), (4, 0.03125, 0.003),
                               (4, 0.234375, 0.0225), (1, 0.5, 1e-6)):
        assert b.dppf_qsr_period(tau_base, beta, lr) == ref.qsr_period(tau_base, f(beta), f(lr))
    assert b.dppf_qsr_period(0, 0.2, 0.1) == -1 and b.dppf_qsr_period(4, 0.2, 0.0) == -1
    mean, pull, push = b.dppf_round_metrics([1.0, 3.0, 8.0], 0.1, 0.5)
    rm, rp, rq = ref.round_metrics([1.0, 3.0, 8.0], f(0.1), f(0.5))
    assert abs(mean - rm) < 1e-6 and push == rq and all(abs(p - q) < 1e-6 for p, q in zip(pull, rp))
    with pytest.raises(b.DppfError):
        b.dppf_round_metrics([1.0, -1.0], 0.1, 0.5)
