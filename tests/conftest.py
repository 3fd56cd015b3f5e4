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
    if not has_gpu:
        skip = pytest.mark.skip(reason="no CUDA device")
        for it in items:
            if "gpu" in it.keywords:
                it.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    # one report of every comparison with the oracle that the session made (tests/parity.py)
    try:
        from tests import parity
        parity.write_report()
    except Exception as e:      # a reporting problem must not change the session's result
        print(f"parity report not written: {e}")
