import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200)")


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
def _checking_build_report(request):
    """Under the checking build (RSLRL_B200_DEBUG_LIBRARY=1) every GPU test ends with its report: no guard
    region next to an allocation overwritten, no out-of-range index recorded."""
    yield
    if os.environ.get("RSLRL_B200_DEBUG_LIBRARY") == "1" and "gpu" in request.node.keywords:
        from paper_2509_10771_b200 import binding
        is_debug, damaged, index_fault = binding.debug_report()
        assert is_debug, "the checking build was asked for but the plain library is loaded"
        assert damaged == 0 and index_fault == 0, (damaged, index_fault)
