import os
import sys
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the library through its C-ABI)")


def pytest_collection_modifyitems(config, items):
    # A GPU test that stalls must fail with the stacks of all threads, not hold the run: every GPU
    # test gets a time limit when the pytest-timeout plug-in is there (the slowest takes ~20 s).
    if config.pluginmanager.hasplugin("timeout"):
        for it in items:
            if "gpu" in it.keywords and it.get_closest_marker("timeout") is None:
                it.add_marker(pytest.mark.timeout(600, method="thread"))
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)
