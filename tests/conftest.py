import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session", autouse=True)
def _oracle_built():
    from oracle.build import build
    build()


@pytest.fixture(scope="session", autouse=True)
def _library_built():
    """libroco.so is built in-tree (and rebuilt when a source is newer); the binding itself never builds."""
    from paper_2402_06262_b200.build import build
    build()
