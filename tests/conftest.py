import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def _have_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    if _have_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """Writes the raw error figures that the parity helpers collected (one JSON object per comparison) to
    parity_errors.jsonl in the report folder (PARITY_REPORT_DIR, default parity_report/ at the repository root);
    tests/parity_report.py turns them into a table."""
    try:
        import json
        import parity_utils
    except Exception:
        return
    if not parity_utils.RECORDS:
        return
    out = os.environ.get("PARITY_REPORT_DIR") or os.path.join(ROOT, "parity_report")
    os.makedirs(out, exist_ok=True)
    with open(os.path.join(out, "parity_errors.jsonl"), "w") as f:
        for r in parity_utils.RECORDS:
            f.write(json.dumps(r) + "\n")
