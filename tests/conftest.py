import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    config.addinivalue_line("markers", "slow: minutes of oracle time; runs only when the -m expression names it (-m 'gpu and slow')")


def pytest_collection_modifyitems(config, items):
    try:
        import torch

        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if "slow" not in (config.getoption("-m") or ""):
        skip_slow = pytest.mark.skip(reason="slow: select it with -m 'gpu and slow'")
        for it in items:
            if "slow" in it.keywords:
                it.add_marker(skip_slow)
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)
