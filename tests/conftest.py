import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def corc():
    """The scalar C oracle."""
    import oracle

    return oracle.c()


@pytest.fixture(scope="session")
def norc():
    """The NumPy oracle."""
    from oracle import oracle_np

    return oracle_np
