import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _guard_bytes_untouched(request):
    """After every GPU test: no kernel wrote outside a buffer the helpers handed out."""
    yield
    if "gpu" in request.keywords:
        import torch
        if torch.cuda.is_available():
            from paper_2511_11248_b200 import helpers
            torch.cuda.synchronize()
            helpers.check_guards(forget=True)
