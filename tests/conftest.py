import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_sessionstart(session):
    """Build the CUDA library (nvcc cross-compiles without a GPU) and the C oracle if they are stale."""
    import shutil
    if shutil.which("nvcc"):
        from paper_2609_28568_b200 import build
        build.build()
    import oracle
    oracle.build()


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
