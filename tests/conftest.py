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


@pytest.fixture(autouse=True)
def _bounds_checked(request):
    """With SCALIFY_DEBUG_BUILD=1 (the bounds-checking build of the library is loaded): every GPU test starts with
    an empty table of registered arrays and fails if the checker refused an access while it ran."""
    if os.environ.get("SCALIFY_DEBUG_BUILD", "") != "1" or "gpu" not in request.keywords:
        yield
        return
    import paper_2407_17353_b200 as sc
    sc.scalify_debug_bounds_report(reset_ranges=True)
    yield
    rep = sc.scalify_debug_bounds_report(reset_ranges=True)
    assert rep["violations"] == 0, rep


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
