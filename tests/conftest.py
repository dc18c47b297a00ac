import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def oracle():
    from oracle.lq_oracle import Oracle
    return Oracle()


@pytest.fixture(scope="session")
def oracle_wide():
    from oracle.lq_oracle import Oracle
    return Oracle(wide=True)


@pytest.fixture(scope="session")
def oracle_plain():
    from oracle.lq_oracle import Oracle
    return Oracle(plain=True)
