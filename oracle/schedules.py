"""Host-side scalars of a DPPF run -- TEST INFRASTRUCTURE ONLY (plain Python, fp64).

* ``lambda_schedule``: the three push-strength schedules of the ablation "How to schedule
  the pushing force?" (appendix): fixed, decreasing lambda/2 (1 + cos(t pi / T)),
  increasing lambda/2 (1 - cos(t pi / T)).
* ``lr_cosine``: cosine annealing of the learning rate, the curve the decreasing schedule
  is said to follow.
* ``qsr_period``: the quadratic synchronisation rule quoted in "Comparison with Other
  Communication-Efficient Methods",
  tau_t = max(tau_base, floor((beta / eta_t)^2)).
* ``round_metrics``: what the pull-push ablation logs per round: the mean worker distance
  (the relaxed Mean Valley measure), the pull strength alpha * r_m and the push strength
  lambda (the push is unit-normed).
"""
import math

FIXED, DECREASING, INCREASING = 0, 1, 2


def lambda_schedule(kind, lam, t, T):
    if kind == FIXED:
        return float(lam)
    c = math.cos(math.pi * t / T)
    if kind == DECREASING:
        return 0.5 * lam * (1.0 + c)
    if kind == INCREASING:
        return 0.5 * lam * (1.0 - c)
    raise ValueError("unknown schedule")


def lr_cosine(lr_max, t, T):
    return 0.5 * lr_max * (1.0 + math.cos(math.pi * t / T))


def qsr_period(tau_base, beta, lr_t):
    return max(int(tau_base), int(math.floor((beta / lr_t) ** 2)))


def round_metrics(norms, alpha, lam):
    norms = [float(r) for r in norms]
    mean_distance = sum(norms) / len(norms)
    pull = [alpha * r for r in norms]
    return mean_distance, pull, float(lam)
