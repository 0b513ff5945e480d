import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # The shared libraries are build outputs, not tracked files: (re)build them when missing or stale
    # (nvcc cross-compiles without a GPU; a few seconds when nothing changed).
    from paper_2104_11981_b200 import build as lib_build
    lib_build.build()
    from oracle import build as oracle_build
    oracle_build.build()


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
