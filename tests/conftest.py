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
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """Writes the achieved parity errors the GPU tests recorded to the file IDKM_PARITY_TABLE names, if any."""
    path = os.environ.get("IDKM_PARITY_TABLE")
    if not path:
        return
    try:
        import parity_util
    except Exception:
        return
    if parity_util.RECORDS:
        parity_util.write_records(path)
