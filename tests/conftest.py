import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
# test_oracle_mutants.py re-runs the pin suite against deliberately broken copies
# of the CPU oracle; it points this variable at the directory holding the copy.
if os.environ.get("DPPF_ORACLE_PARENT"):
    sys.path.insert(0, os.environ["DPPF_ORACLE_PARENT"])


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle
