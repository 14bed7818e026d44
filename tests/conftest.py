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


def pytest_sessionfinish(session, exitstatus):
    """Writes the unscaled error figures the parity tests collected (tests/parity_utils.REPORT) to the
    file named by LRSA_PARITY_REPORT, one JSON record per comparison."""
    path = os.environ.get("LRSA_PARITY_REPORT")
    mod = sys.modules.get("tests.parity_utils")
    if not path or mod is None or not mod.REPORT:
        return
    import json
    with open(path, "w") as f:
        for rec in mod.REPORT:
            f.write(json.dumps(rec) + "\n")
