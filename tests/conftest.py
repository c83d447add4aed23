import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """The CUDA library, compiled once per session when its sources are newer than the binary (nvcc
    cross-compiles for sm_100a without a GPU); tests that load it must not depend on collection order."""
    from paper_2411_00288_b200 import build as libbuild
    libbuild.build()
