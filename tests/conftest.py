import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def tiny_wl():
    from gen import configs
    return configs.tiny()


@pytest.fixture(scope="session")
def small_wl():
    from gen import configs
    return configs.small()
