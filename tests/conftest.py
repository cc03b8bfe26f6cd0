import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a library)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(autouse=True)
def output_guards(request):
    """GPU tests: every output tensor the binding creates sits between guard zones, verified after the test (the
    stand-in for a memory checker: a kernel that writes just outside an output fails the test that ran it)."""
    if "gpu" not in request.keywords:
        yield
        return
    import paper_1804_02941_b200 as d
    d.guards_enable(True)
    try:
        yield
        d.guards_check()
    finally:
        d.guards_enable(False)
