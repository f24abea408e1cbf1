import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")


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
def _guard_bytes_intact(request):
    """After every GPU test: no kernel wrote past the end of a device block (256 guard bytes follow each block of
    every cache; lq_check_guards).  Caches closed inside the test are checked by close() itself."""
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2503_19950_b200 import LogQuantCache
    LogQuantCache.guards_on_close = True
    yield
    for cache in list(LogQuantCache.live):
        if getattr(cache, "_h", None) and cache.cfg.device >= 0:
            assert cache.check_guards() == 0, "a kernel wrote past the end of a device block"
