import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(autouse=True)
def guard_bands(request, monkeypatch):
    """Memory-safety evidence for the GPU tests: every device block the binding hands to the library
    (descriptor table, cache slab, workspace) is carved out of a larger block with a patterned band on
    both sides; after the test the bands must be intact.  A kernel that writes outside its block fails
    the test that ran it."""
    if "gpu" not in request.keywords:
        yield
        return
    import torch
    if not torch.cuda.is_available():
        yield
        return
    from paper_2311_04951_b200 import binding
    from tests import gpu_util
    reg = gpu_util.GuardedAllocator()
    monkeypatch.setattr(binding, "device_buffer", reg.alloc)
    yield reg
    torch.cuda.synchronize()
    reg.check()
