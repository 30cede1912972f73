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
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _guard_bands(request):
    """GPU tests: every buffer the binding allocates is poisoned and sits between guard bands, which are
    checked when the test ends (the stand-in for a memory checker on the kernels' stores)."""
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2506_04985_b200 import binding
    import helpers
    helpers.GUARDS.live = []
    binding.set_allocator(helpers.GUARDS)
    try:
        yield
        import torch
        torch.cuda.synchronize()
        helpers.GUARDS.check(release=True)
    finally:
        helpers.GUARDS.live = []
        binding.set_allocator(None)
