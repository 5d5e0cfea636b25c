import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")
    config.addinivalue_line("markers", "slow: long-running case, enabled with KV_SLOW=1")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have_gpu = False
    skip_gpu = pytest.mark.skip(reason="no CUDA device")
    skip_slow = pytest.mark.skip(reason="set KV_SLOW=1 to run")
    for item in items:
        if "gpu" in item.keywords and not have_gpu:
            item.add_marker(skip_gpu)
        if "slow" in item.keywords and os.environ.get("KV_SLOW") != "1":
            item.add_marker(skip_slow)
