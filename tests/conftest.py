import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import ffd_oracle
    ffd_oracle.set_threads(min(8, ffd_oracle.max_threads()))
    return ffd_oracle
