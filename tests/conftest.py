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


@pytest.fixture(autouse=True)
def _checked_build_reports_nothing(request):
    """Under HYENAND_LIB=debug (the library compiled with range checks on every global-memory access) each GPU test
    also requires that no kernel touched an address outside the tensors and allocations of its call."""
    yield
    if os.environ.get("HYENAND_LIB") != "debug" or "gpu" not in request.keywords:
        return
    from paper_2607_19378_b200 import hyenand as H
    if not H.hyenand_debug_build():
        pytest.fail("HYENAND_LIB=debug did not load the checked build")
    n, addr, line, name = H.hyenand_debug_violations()
    assert n == 0, f"{n} accesses outside the call's ranges; first at {addr:#x}, {name}:{line}"
