import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session", autouse=True)
def built_library():
    """Builds the CUDA library in-tree when it is missing or older than its sources (nvcc
    cross-compiles without a GPU).  A failed build fails the session: nothing stands in for it."""
    from paper_2505_10183_b200 import build
    if build.is_stale():
        build.build()
    return build.LIB


@pytest.fixture(scope="session")
def oracle():
    from oracle import kt_oracle
    kt_oracle.lib()
    return kt_oracle
