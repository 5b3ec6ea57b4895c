import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle_mod():
    import oracle
    return oracle


@pytest.fixture(scope="session")
def code_2_2(oracle_mod):
    return oracle_mod.Code(2, 2)


@pytest.fixture(scope="session")
def code_3_3(oracle_mod):
    return oracle_mod.Code(3, 3)


@pytest.fixture(scope="session")
def code_2_13(oracle_mod):
    return oracle_mod.Code(2, 13)


@pytest.fixture(scope="session")
def code_2_53(oracle_mod):
    return oracle_mod.Code(2, 53)
