import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def golden_dir():
    return ROOT / "tests" / "golden"


@pytest.fixture(scope="session", autouse=True)
def _built_libraries():
    """Compile the CUDA library (nvcc cross-compiles without a GPU) and the C oracle once."""
    from paper_2608_09291_b200 import build as libbuild
    import oracle
    libbuild.build()
    oracle.build()
