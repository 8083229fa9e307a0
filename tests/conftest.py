import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """The C-ABI library and the C part of the oracle are built in-tree before any test (a no-op when they are fresh)."""
    from paper_2601_16032_b200 import build as lib_build
    from oracle import build as oracle_build
    lib_build.build()
    oracle_build.build()
