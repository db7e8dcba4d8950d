import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


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
    """Writes the audit table of the end-to-end comparisons (tests/gpu_util.check_e2e) to $METIS_PARITY_LOG."""
    path = os.environ.get("METIS_PARITY_LOG")
    try:
        import gpu_util
    except Exception:
        return
    if not path or not gpu_util.E2E_RECORDS:
        return
    with open(path, "w") as f:
        f.write("# case | errors | allowance added to 2e-3 | differing factor blocks / all | plain 2e-3 held\n")
        for r in gpu_util.E2E_RECORDS:
            f.write("%s | %s | %.2e | %d/%d | %s\n" % (r["case"], " ".join("%s=%.3e" % kv for kv in r["errors"].items()),
                                                     r["allowance"], r["differing_blocks"], r["factor_blocks"],
                                                     "yes" if r["plain_tolerance_held"] else "no"))
