import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_addoption(parser):
    parser.addoption("--run-slow", action="store_true", default=False,
                     help="also run the tests marked slow (workloads at their full stated extent: minutes of GPU and host time)")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200 box)")
    config.addinivalue_line("markers", "slow: full-extent workloads that take minutes; run with --run-slow or SKIPKV_RUN_SLOW=1")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    run_slow = config.getoption("--run-slow") or os.environ.get("SKIPKV_RUN_SLOW") == "1"
    skip_gpu = pytest.mark.skip(reason="no CUDA device")
    skip_slow = pytest.mark.skip(reason="slow: run with --run-slow or SKIPKV_RUN_SLOW=1")
    for item in items:
        if "gpu" in item.keywords and not has_gpu:
            item.add_marker(skip_gpu)
        if "slow" in item.keywords and not run_slow:
            item.add_marker(skip_slow)
