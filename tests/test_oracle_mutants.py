"""The pin suite must notice a plausible slip anywhere in the CPU oracle.

Each case copies ``oracle/`` to a scratch directory, plants one textual mistake in
the C source (CPU only), and re-runs ``test_oracle_pins.py`` against the copy in a
child process; the run has to fail."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MUTANTS = {
    "control_unchanged": ("", ""),
    "push_sign": ("a - lam / r_out[m]", "a + lam / r_out[m]"),
    "direction": ("(A[i] - xi) * c", "(xi - A[i]) * c"),
    "mean_divisor": ("A[i] = s / (double)M;", "A[i] = s / (double)(M > 1 ? M - 1 : 1);"),
    "no_sqrt": ("r_out[m] = sqrt(S);", "r_out[m] = S;"),
    "not_squared": ("S += diff * diff;", "S += diff;"),
    "row_stride": ("const float *xm = x + (int64_t)m * ld;", "const float *xm = x + (int64_t)m * d;"),
    "pull_weight": ("y[i] = (1.0 - a) * xi + a * A[i];", "y[i] = (1.0 - a) * A[i] + a * xi;"),
    "momentum_sign": ("vm[i] = mu * vm[i] + gt;", "vm[i] = mu * vm[i] - gt;"),
    "decay_operand": ("(double)gm[i] + wd * xm[i];", "(double)gm[i] + wd * vm[i];"),
    "descent_sign": ("xm[i] = xm[i] - eta * vm[i];", "xm[i] = xm[i] + eta * vm[i];"),
    "f64_round_coeff": ("(float)(xm[i] + (A[i] - xm[i]) * c)", "(float)(xm[i] + (A[i] - xm[i]) * a)"),
    "adamw_decay": ("xw[i] = xw[i] * (1.0 - eta * wd);", "xw[i] = xw[i] * (1.0 - wd);"),
    "adamw_second_moment": ("(1.0 - b2) * gi * gi;", "(1.0 - b2) * gi;"),
    "adamw_bias": ("sqrt(bw[i] / bc2) + e", "sqrt(bw[i]) + e"),
    # general round
    "g_push_reference": ("double dn = y - P[i];", "double dn = y - A[i];"),
    "g_weight_norm": ("C[i] = c / wsum;", "C[i] = c;"),
    "g_mean_direction": ("for (int64_t i = 0; i < d; ++i) ubar[i] /= (double)M;", ""),
    "g_second_term_sign": ("lam * (u - ubar[i])", "lam * (u + ubar[i])"),
    "g_pull_target": ("double y = (1.0 - a) * (double)xm[i] + a * C[i];\n            double u =",
                      "double y = (1.0 - a) * (double)xm[i] + a * A[i];\n            double u ="),
    "g_distance_reference": ("double dr = xi - A[i];", "double dr = xi - C[i];"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_mutant(tmp_path, name):
    old, new = MUTANTS[name]
    dst = tmp_path / "oracle"
    shutil.copytree(os.path.join(ROOT, "oracle"), dst,
                    ignore=shutil.ignore_patterns("*.so", "__pycache__", "*.tmp*"))
    src = (dst / "dppf_oracle.c").read_text()
    assert old in src, f"mutation site for {name} not found"
    (dst / "dppf_oracle.c").write_text(src.replace(old, new))
    env = dict(os.environ, DPPF_ORACLE_PARENT=str(tmp_path))
    files = [os.path.join(ROOT, "tests", "test_oracle_pins.py"),
             os.path.join(ROOT, "tests", "test_oracle_general_pins.py")]
    if name.startswith("g_"):
        files.reverse()                      # the suite that should notice goes first (-x stops there)
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", *files],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    if name == "control_unchanged":          # the copy mechanism itself must not break the suite
        assert run.returncode == 0, run.stdout[-2000:]
        return
    assert run.returncode == 1, f"mutant {name} survived:\n{run.stdout[-2000:]}"
