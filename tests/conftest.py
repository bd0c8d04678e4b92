import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def orc():
    """The CPU oracle, compiled on first use."""
    import oracle
    oracle.build()
    return oracle


_WL_CACHE = {}


@pytest.fixture(scope="session")
def workloads():
    """Session cache of generated workloads keyed by config name."""
    from paper_2607_06202_b200 import workload as W

    def get(name):
        if name not in _WL_CACHE:
            _WL_CACHE[name] = W.make_workload(W.CONFIGS[name])
        return _WL_CACHE[name]
    return get
