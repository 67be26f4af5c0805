import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _index_checks_stay_clean(request):
    """When the suite runs on the index-check build of the library (ROBE_LIBRARY names it), every GPU
    test must leave the library's debug word at zero: no kernel computed an index beyond its bound."""
    yield
    if "gpu" in request.keywords and os.environ.get("ROBE_LIBRARY"):
        import paper_2108_02191_b200 as robe
        code = robe.robe_debug_status()
        assert code == 0, f"a kernel of the index-check build failed check {code} (ROBE_DBG_* in include/robe.h)"
