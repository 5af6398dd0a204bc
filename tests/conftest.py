import os
import sys

# The oracle's numpy code runs on the host next to other jobs: a bounded BLAS thread pool keeps its
# spin-waiting threads from multiplying the slowdown when the host cores are oversubscribed.
for _v in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS"):
    os.environ.setdefault(_v, "8")

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
                it.add_marker(pytest.mark.timeout(int(os.environ.get("RPO_GPU_TEST_TIMEOUT", "600")), method="thread"))
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
