import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _tolerance_use(request, record_property):
    """Attaches to every test the largest error each of its tolerance checks saw and the share of the
    tolerance it used (shown by `pytest -rA`; written to the file named by SAR_TOL_REPORT, if set)."""
    import helpers
    helpers.TOLERANCE_USE.clear()
    yield
    rows = list(helpers.TOLERANCE_USE)
    helpers.TOLERANCE_USE.clear()
    if not rows:
        return
    text = "; ".join(f"{w}: err {e:.2e} = {100 * u:.0f}% of tol" for w, e, u in rows)
    record_property("tolerance_use", text)
    print("tolerance use: " + text)
    path = os.environ.get("SAR_TOL_REPORT")
    if path:
        with open(path, "a") as fh:
            fh.write(f"{request.node.nodeid}\t{text}\n")
