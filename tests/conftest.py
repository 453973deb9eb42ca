import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_sessionfinish(session, exitstatus):
    """DES_TOL_REPORT=<file>: write how many compared elements needed more than the stated
    1e-5 relative / 1e-6 absolute bound (tests/harness.py: TOL_STATS), per output."""
    path = os.environ.get("DES_TOL_REPORT")
    if not path:
        return
    try:
        import json
        import harness
        with open(path, "w") as f:
            json.dump(harness.TOL_STATS, f, indent=1, sort_keys=True)
    except Exception as e:   # a report, not a test
        print(f"tolerance report not written: {e!r}")
