import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_sessionfinish(session, exitstatus):
    """With XY_PARITY_REPORT=<file> set, leaves the largest parity errors seen in this session there."""
    path = os.environ.get("XY_PARITY_REPORT")
    if not path:
        return
    try:
        import json

        from tests import helpers as H
        if H.OBSERVED["checks"]:
            with open(path, "w") as f:
                json.dump(H.OBSERVED, f)
    except Exception:
        pass
