"""Shared pytest set-up: the ``gpu`` marker and paths."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN_DIR = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def golden_dir():
    return GOLDEN_DIR


def pytest_sessionfinish(session, exitstatus):
    """With AKG_PARITY_LOG=<file>: how many elements of each slack-widened comparison needed the slack."""
    path = os.environ.get("AKG_PARITY_LOG")
    if not path:
        return
    try:
        import parity_util
    except Exception:
        return
    with open(path, "w") as fh:
        total = sum(r for _, _, r in parity_util.RESCUE_LOG)
        fh.write(f"# comparisons with a slack: {len(parity_util.RESCUE_LOG)}, elements rescued: {total}\n")
        for what, n, rescued in parity_util.RESCUE_LOG:
            if rescued:
                fh.write(f"{rescued}\t{n}\t{what}\n")
