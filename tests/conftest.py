import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


_build_error = None


def pytest_configure(config):
    global _build_error
    config.addinivalue_line("markers", "gpu: needs a CUDA device and the built library")
    from paper_2307_02628_b200 import build
    try:
        build.build()        # no-op when libskipdecode.so is newer than its sources
    except RuntimeError as e:    # no nvcc here: the oracle's own pins still run, what needs the library fails by itself
        _build_error = str(e)


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device" + (f"; library not built: {_build_error}" if _build_error else ""))
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session")
def repo_root():
    return ROOT
