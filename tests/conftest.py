import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); runs the library through its C ABI")
    config.addinivalue_line("markers", "soak: long opt-in GPU checks (fuzz, > 4 GB tensors, repeated steps); run with -m soak")


def _have_gpu() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    # the long checks run only when asked for by name (-m soak), never as part of "-m gpu" or "-m 'not gpu'"
    if "soak" not in (config.getoption("-m") or ""):
        skip_soak = pytest.mark.skip(reason="opt-in: run with -m soak")
        for item in items:
            if "soak" in item.keywords:
                item.add_marker(skip_soak)
    if _have_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords or "soak" in item.keywords:
            item.add_marker(skip)
