import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")


@pytest.fixture(scope="session")
def oracle64():
    from oracle.kge_oracle import Oracle
    return Oracle("f64")


@pytest.fixture(scope="session")
def oracle32():
    from oracle.kge_oracle import Oracle
    return Oracle("f32")


@pytest.fixture(scope="session")
def oracle64_tie():
    """The fp64 oracle built with sign(0) = -1 as the sub-gradient of |x| at an exact tie."""
    from oracle.kge_oracle import Oracle
    return Oracle("f64_tie")
