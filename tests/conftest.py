import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # the tests import the ctypes binding at collection time: make sure the library exists
    from paper_1603_06809_b200.build import ensure_built
    ensure_built()


@pytest.fixture(scope="session")
def oracle():
    from oracle import bcast_oracle
    bcast_oracle.build()
    return bcast_oracle
