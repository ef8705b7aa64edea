"""Shared helpers for the GPU parity tests (upload / download / tolerance checks)."""
import numpy as np


def require_gpu():
    import torch
    if not torch.cuda.is_available():
        import pytest
        pytest.skip("no CUDA device")
    from paper_2507_20424_b200 import binding
    binding.load(rebuild_if_stale=True)   # compiles with nvcc if needed; raises if it cannot: no fallback
    return torch, binding


def to_dev(a):
    import torch
    return torch.from_numpy(a).cuda()


def padded(x, d=None):
    """Copy of x[M, d] in an [M, ld] array whose pad columns are NaN."""
    from paper_2507_20424_b200 import inputs
    M, d0 = x.shape
    d = d0 if d is None else d
    out = inputs.empty_rows(M, d)
    out[:, :d] = x[:, :d]
    return out


# tolerances stated for the method: |dx| <= 1e-6 (1 + |x|) per element, 1e-5 relative on norms
def assert_parity(x_gpu, r_gpu, x_ref, r_ref, d):
    x_ref = x_ref[:, :d].astype(np.float64)
    err = np.abs(x_gpu[:, :d].astype(np.float64) - x_ref)
    bound = 1e-6 * (1.0 + np.abs(x_ref))
    assert np.all(err <= bound), f"max excess {np.max(err - bound):.3e}, max err {err.max():.3e}"
    r_ref = np.asarray(r_ref, dtype=np.float64)
    r_gpu = np.asarray(r_gpu, dtype=np.float64)
    assert np.all(np.abs(r_gpu - r_ref) <= 1e-5 * r_ref), (r_gpu, r_ref)
    assert np.all(r_gpu[r_ref == 0.0] == 0.0)


def assert_pad_untouched(a, d):
    if a.shape[1] > d:
        assert np.all(np.isnan(a[:, d:])), "pad columns were written"


def same_bits(a, b):
    return np.array_equal(a.view(np.uint32), b.view(np.uint32))
