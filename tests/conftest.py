import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); deselected on CPU-only hosts")


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
def _guard_bands(request):
    """GPU tests: every tensor the binding allocates for the library (outputs, accumulator dumps, workspaces) gets
    canary bands on both sides, checked when the test ends."""
    if "gpu" not in request.keywords:
        yield
        return
    import torch
    if not torch.cuda.is_available():
        yield
        return
    from helpers import GuardedAllocator
    from paper_2605_13915_b200 import binding
    g = GuardedAllocator()
    old = (binding._empty, binding._workspace)
    binding._empty, binding._workspace = g.empty, g.workspace
    try:
        yield
        g.check()
    finally:
        binding._empty, binding._workspace = old
        binding.debug_reset_options()        # a test may have forced a schedule (msd_debug_set_option)
