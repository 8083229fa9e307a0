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


def nvcc_available() -> bool:
    import shutil
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return os.path.exists(nvcc) or shutil.which(nvcc) is not None


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """The C part of the oracle is built in-tree before any test; so is the C-ABI library where nvcc exists (both are
    no-ops when fresh).  Without nvcc the oracle's own pins still run; the tests that load the CUDA library skip."""
    from oracle import build as oracle_build
    oracle_build.build()
    if nvcc_available():
        from paper_2601_16032_b200 import build as lib_build
        lib_build.build()
