import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


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
    """With SCALIFY_TOLERANCE_LOG=<file>: per test function, how many outputs were compared by
    helpers.within() and how many of them only its cancellation clause accepted."""
    path = os.environ.get("SCALIFY_TOLERANCE_LOG")
    if not path:
        return
    try:
        import helpers
    except Exception:
        return
    totals = {}
    for label, n, n_loose in helpers.LOOSE_LOG:
        t = totals.setdefault(label, [0, 0, 0.0])
        t[0] += n
        t[1] += n_loose
        t[2] = max(t[2], n_loose / max(n, 1))
    with open(path, "w") as f:
        f.write("# test function, outputs compared, accepted only by the cancellation clause, share, largest share in one call\n")
        for label in sorted(totals):
            n, nl, worst = totals[label]
            f.write(f"{label}\t{n}\t{nl}\t{nl / max(n, 1):.3e}\t{worst:.3e}\n")
