import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


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


@pytest.fixture(autouse=True)
def _no_access_outside_its_buffer(request):
    """Under the bounds-checked build (MXQ_LIBRARY=checked) every GPU test also asserts that no kernel of the linear
    path formed an address outside the buffer it belongs to (the test that provokes one on purpose reads the report
    itself)."""
    yield
    if os.environ.get("MXQ_LIBRARY") != "checked" or "gpu" not in request.keywords:
        return
    import paper_2503_13565_b200 as mxq
    report = mxq.mxq_debug_bounds_report()
    assert report["checked"] and report["refused"] == 0, report
