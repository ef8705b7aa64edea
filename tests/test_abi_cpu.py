"""Host-side checks that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_20424_b200 import binding, build
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dppf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dppf_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2507_20424_b200 import binding
    names = declared_symbols()
    assert "dppf_consensus" in names and "dppf_local_step_and_consensus" in names
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_workspace_bytes(lib):
    from paper_2507_20424_b200 import binding
    assert binding.workspace_bytes(0, 10) == 0 and binding.workspace_bytes(4, 0) == 0
    assert binding.workspace_bytes(1025, 10) == 0
    w4, w16, w64 = (binding.workspace_bytes(m, 10**6) for m in (4, 16, 64))
    assert 0 < w4 < w16 and w64 > 0 and all(w % 256 == 0 for w in (w4, w16, w64))


def test_status_strings(lib):
    from paper_2507_20424_b200 import binding
    assert [binding.status_string(i) for i in range(6)] == [
        "DPPF_OK", "DPPF_ERR_INVALID_ARG", "DPPF_ERR_ALIGNMENT", "DPPF_ERR_WORKSPACE",
        "DPPF_ERR_CUDA", "DPPF_ERR_TIMEOUT"]
    assert binding.status_string(99) == "DPPF_ERR_UNKNOWN"


def test_launch_count(lib):
    from paper_2507_20424_b200 import binding as b
    assert b.launch_count(4, 100, b.PATH_TWO_KERNEL) == 2
    assert b.launch_count(4, 100, b.PATH_COOPERATIVE) == 1
    assert b.launch_count(64, 100, b.PATH_COOPERATIVE) == 2      # generic kernels: two launches
    assert b.launch_count(1, 100) == 1 and b.launch_count(1, 100, fused=True) == 2
    assert b.launch_count(0, 100) == 0


def test_argument_validation_happens_before_any_cuda_call(lib):
    """Fake but well-formed pointers: every call must be rejected on the host."""
    from paper_2507_20424_b200 import binding as b
    X, V, G, WS = 0x10000000, 0x20000000, 0x30000000, 0x40000000
    big = 1 << 30
    f = lib.dppf_consensus
    assert f(None, 4, 64, 64, 0.1, 0.01, None, WS, big, None) == b.ERR_INVALID_ARG
    assert f(X, 0, 64, 64, 0.1, 0.01, None, WS, big, None) == b.ERR_INVALID_ARG
    assert f(X, 4, 0, 64, 0.1, 0.01, None, WS, big, None) == b.ERR_INVALID_ARG
    assert f(X, 4, 65, 64, 0.1, 0.01, None, WS, big, None) == b.ERR_INVALID_ARG      # ld < d
    assert f(X, 4, 60, 60, 0.1, 0.01, None, WS, big, None) == b.ERR_ALIGNMENT        # ld % 32
    assert f(X + 4, 4, 64, 64, 0.1, 0.01, None, WS, big, None) == b.ERR_ALIGNMENT
    assert f(X, 4, 64, 64, float("nan"), 0.01, None, WS, big, None) == b.ERR_INVALID_ARG
    assert f(X, 4, 64, 64, 0.1, float("inf"), None, WS, big, None) == b.ERR_INVALID_ARG
    assert f(X, 4, 64, 64, 0.1, 0.01, None, None, big, None) == b.ERR_INVALID_ARG
    assert f(X, 4, 64, 64, 0.1, 0.01, None, WS, 16, None) == b.ERR_WORKSPACE
    assert f(X, 4, 64, 64, 0.1, 0.01, None, X + 512, big, None) == b.ERR_INVALID_ARG  # ws inside x
    assert lib.dppf_consensus_ex(X, 4, 64, 64, 0.1, 0.01, None, WS, big, 7, None) == b.ERR_INVALID_ARG
    g = lib.dppf_local_step
    assert g(X, None, G, 4, 64, 64, 0.1, 0.9, 1e-4, None) == b.ERR_INVALID_ARG
    assert g(X, X, G, 4, 64, 64, 0.1, 0.9, 1e-4, None) == b.ERR_INVALID_ARG           # x aliases v
    assert g(X, V, G, 4, 64, 64, float("nan"), 0.9, 1e-4, None) == b.ERR_INVALID_ARG
    h = lib.dppf_local_step_and_consensus
    assert h(X, V, V + 128, 4, 64, 64, 0.1, 0.9, 1e-4, 0.1, 0.01, None, WS, big, None) == b.ERR_INVALID_ARG
    assert h(X, V, G, 4, 64, 64, 0.1, 0.9, 1e-4, 0.1, 0.01, None, WS, 16, None) == b.ERR_WORKSPACE
    k = lib.dppf_consensus_host
    assert k(None, 4, 64, 64, 0.1, 0.01, None, X, WS, big, None) == b.ERR_INVALID_ARG
    assert k(V, 4, 64, 64, 0.1, 0.01, None, X + 4, WS, big, None) == b.ERR_ALIGNMENT
    assert lib.dppf_device_status(None, None) == b.ERR_INVALID_ARG
    assert lib.dppf_device_schedule(None, None) == b.ERR_INVALID_ARG
    gen = lib.dppf_consensus_general
    w_ok = (ctypes.c_float * 4)(1, 2, 3, 4)
    w_zero = (ctypes.c_float * 4)(0, 0, 0, 0)
    assert gen(None, 4, 64, 64, 0.1, 0.01, None, 0, 0, None, None, WS, big, None) == b.ERR_INVALID_ARG
    assert gen(X, 17, 64, 64, 0.1, 0.01, None, 0, 0, None, None, WS, big, None) == b.ERR_INVALID_ARG
    assert gen(X, 4, 64, 64, 0.1, 0.01, w_ok, 2, 0, None, None, WS, big, None) == b.ERR_INVALID_ARG
    assert gen(X, 4, 64, 64, 0.1, 0.01, w_zero, 0, 0, None, None, WS, big, None) == b.ERR_INVALID_ARG
    assert gen(X, 4, 64, 64, 0.1, 0.01, w_ok, 0, 1, None, None, WS, 16, None) == b.ERR_WORKSPACE
    assert gen(X, 4, 60, 60, 0.1, 0.01, w_ok, 0, 1, None, None, WS, big, None) == b.ERR_ALIGNMENT
    rounds = lib.dppf_consensus_rounds
    lam_bad = (ctypes.c_float * 2)(0.1, float("inf"))
    assert rounds(None, 4, 64, 64, 0.1, 0.01, None, 3, None, WS, big, None) == b.ERR_INVALID_ARG
    assert rounds(X, 4, 64, 64, 0.1, 0.01, None, 0, None, WS, big, None) == b.ERR_INVALID_ARG
    assert rounds(X, 4, 64, 64, 0.1, 0.01, lam_bad, 2, None, WS, big, None) == b.ERR_INVALID_ARG
    assert rounds(X, 4, 64, 64, float("nan"), 0.01, None, 2, None, WS, big, None) == b.ERR_INVALID_ARG
    assert rounds(X, 4, 64, 64, 0.1, 0.01, None, 2, None, WS, 16, None) == b.ERR_WORKSPACE
    assert rounds(X, 4, 64, 64, 0.1, 0.01, None, 2, X + 64, WS, big, None) == b.ERR_INVALID_ARG   # norms inside x
    SUMS = 0x50000000
    dp, uf = lib.dppf_distance_partials, lib.dppf_update_from_sums
    assert dp(None, 4, 64, 64, SUMS, WS, big, None) == b.ERR_INVALID_ARG
    assert dp(X, 4, 64, 64, None, WS, big, None) == b.ERR_INVALID_ARG
    assert dp(X, 4, 64, 64, SUMS + 4, WS, big, None) == b.ERR_INVALID_ARG             # fp64 alignment
    assert dp(X, 4, 64, 64, SUMS, WS, 16, None) == b.ERR_WORKSPACE
    assert dp(X, 4, 64, 64, X + 8, WS, big, None) == b.ERR_INVALID_ARG                # sums inside x
    assert uf(X, 4, 64, 64, 0.1, 0.01, None, None, None) == b.ERR_INVALID_ARG
    assert uf(X, 4, 64, 64, float("inf"), 0.01, SUMS, None, None) == b.ERR_INVALID_ARG
    assert uf(X, 4, 60, 60, 0.1, 0.01, SUMS, None, None) == b.ERR_ALIGNMENT
    assert lib.dppf_consensus_general_ex(X, 4, 64, 64, 0.1, 0.01, None, 0, 0, None, None, WS, big, 2, None) == b.ERR_INVALID_ARG
    assert lib.dppf_consensus_static(X, 4, 64, 64, float("nan"), 0.01, None, None) == b.ERR_INVALID_ARG
    assert lib.dppf_consensus_rounds_ex(X, 4, 64, 64, 0.1, 0.01, None, 2, None, WS, big, 9, None) == b.ERR_INVALID_ARG


def test_binding_refuses_cpu_tensors(lib):
    import torch
    from paper_2507_20424_b200 import binding
    with pytest.raises(ValueError):
        binding.dppf_consensus(torch.zeros(4, 64), 0.1, 0.01)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2507_20424_b200 import binding, build
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(build, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
