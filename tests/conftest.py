import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (parity of the CUDA path against the oracle)")


def pytest_collection_modifyitems(config, items):
    # GPU tests are skipped, not failed, where no device exists and the run did not ask for them.
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
    # Under the bounds-check build (ARB_LIB_VARIANT=checks) the buffers of the shared context lie between guard
    # zones: after the last test they must still hold their pattern.
    if os.environ.get("ARB_LIB_VARIANT") != "checks":
        return
    from tests import helpers
    bad, checked = helpers.guard_zones()
    print(f"\nguard zones: {checked} bytes checked, {bad} overwritten")
    if bad and session.exitstatus == 0:
        session.exitstatus = 1
