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
    from oracle import lla_oracle
    lla_oracle.build()
    return lla_oracle


@pytest.fixture(scope="session")
def backward_oracle():
    from oracle import lla_backward_oracle
    return lla_backward_oracle
