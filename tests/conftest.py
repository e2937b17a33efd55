import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


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
def _guard_bands(request):
    """GPU tests give every cache 64 KiB of patterned guard band on either side of its arena and of
    its workspace (a stand-in for a memory checker): `close()` raises when a kernel wrote there, and
    caches a test leaves open are checked when the test ends."""
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2508_12407_b200 import binding
    live = []
    orig_init = binding.ZigzagCache.__init__

    def tracking_init(self, *a, **kw):
        orig_init(self, *a, **kw)
        live.append(self)

    binding.ZigzagCache.default_guard_bytes = 64 * 1024
    binding.ZigzagCache.__init__ = tracking_init
    try:
        yield
    finally:
        binding.ZigzagCache.__init__ = orig_init
        binding.ZigzagCache.default_guard_bytes = 0
    for c in live:
        if getattr(c, "_h", None):
            assert c.guards_intact(), "a kernel wrote outside the arena or the workspace"
