import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_sessionstart(session):
    """Build the CUDA library (nvcc cross-compiles without a GPU) and the C oracle when they are
    missing or older than their sources, so that a fresh checkout can run the suite directly."""
    from paper_2609_32999_b200 import build as lib_build
    from oracle import tessera_oracle
    try:
        lib_build.build()
    except Exception:
        if not os.path.exists(lib_build.LIB):      # no library at all: nothing can run
            raise
    tessera_oracle.build()


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has = torch.cuda.is_available()
    except Exception:
        has = False
    if has:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)
