import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device and the built library")
    from paper_2307_02628_b200 import build
    build.build()            # no-op when libskipdecode.so is newer than its sources


@pytest.fixture(scope="session")
def repo_root():
    return ROOT
