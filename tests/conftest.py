import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle_lib():
    import oracle

    oracle.build()
    return oracle


@pytest.fixture(scope="session")
def s4c_lib():
    """The built C-ABI library path (compiles it in-tree with nvcc if it is missing or stale)."""
    import paper_2506_14158_b200 as pkg

    pkg.build()
    return pkg.lib_path()
