import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
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


@pytest.fixture(autouse=True)
def _release_device_memory(request):
    """After every GPU test: hand cached device memory back, so that the full-size tests that
    follow (they check how much is free before they start) see the whole GPU."""
    yield
    if "gpu" in request.keywords:
        import gc
        import torch
        if torch.cuda.is_available():
            gc.collect()
            torch.cuda.empty_cache()
