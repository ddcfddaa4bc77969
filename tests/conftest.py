import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Builds the CUDA library and the CPU checker if they are missing or older than their sources (a no-op
    otherwise), so that a fresh checkout can run the tests directly."""
    from oracle import build as oracle_build
    from paper_2605_01989_b200 import build as lib_build
    lib_build.build()
    oracle_build.build()
