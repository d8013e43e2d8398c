import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


GPU_TEST_SECONDS = 300   # a GPU test that runs longer than this is ended with its process


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200)")
    if not config.pluginmanager.hasplugin("timeout"):
        config.addinivalue_line("markers", "timeout: per-test time limit (pytest-timeout, when installed)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        # every device wait in the kernels is bounded, so no test should ever get here; if one does
        # (a kernel that never returns cannot be interrupted by a signal), the process is ended
        for item in items:
            if "gpu" in item.keywords and item.get_closest_marker("timeout") is None:
                item.add_marker(pytest.mark.timeout(GPU_TEST_SECONDS, method="thread"))
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
