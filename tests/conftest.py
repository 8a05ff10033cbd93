import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


def pytest_sessionfinish(session, exitstatus):
    """The parity statistics of a GPU run (flipped and adopted codes, their fractions and margins) go to
    parity_stats.json in the directory PARITY_STATS_DIR names, when it is set."""
    out_dir = os.environ.get("PARITY_STATS_DIR")
    try:
        import parity
    except Exception:
        return
    if out_dir and parity.ALL_STATS:
        import json
        os.makedirs(out_dir, exist_ok=True)
        with open(os.path.join(out_dir, "parity_stats.json"), "w") as f:
            json.dump(parity.ALL_STATS, f, indent=1)
