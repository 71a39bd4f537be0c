import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built library")


@pytest.fixture(scope="session")
def oracle():
    """The fp64 CPU oracle, compiled on first use."""
    from oracle import zsm_oracle
    zsm_oracle.build()
    return zsm_oracle
