import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle (compiled on first use)."""
    from oracle import ahakv_oracle
    ahakv_oracle.build()
    return ahakv_oracle


def golden_path(name):
    return os.path.join(ROOT, "tests", "golden", name)
