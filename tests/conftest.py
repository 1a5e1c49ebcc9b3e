import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _o
    _o.lib()
    return _o


def pytest_sessionfinish(session, exitstatus):
    """With HQ_PARITY_STATS=<file>, the measured mismatch fractions and tie distances of the code comparisons are
    written there as JSON lines (the figures the tolerances of the normalisation prologues are set from)."""
    path = os.environ.get("HQ_PARITY_STATS")
    if not path:
        return
    import json
    try:
        from hq_testutil import PARITY_STATS
    except ImportError:
        return
    with open(path, "w") as f:
        for rec in PARITY_STATS:
            f.write(json.dumps(rec) + "\n")
