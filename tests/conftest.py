import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


_NEEDS_LIBRARY = False


@pytest.fixture(scope="session", autouse=True)
def _library_is_built():
    """libolsgd.so is built in-tree before the GPU tests run (a no-op when it is up to date).
    Sessions that only exercise the CPU oracle do not build: they need no nvcc.  The host-side
    ABI tests build through their own fixture."""
    if _NEEDS_LIBRARY:
        from paper_2002_09539_b200.build import build
        build()


def pytest_collection_modifyitems(config, items):
    global _NEEDS_LIBRARY
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        _NEEDS_LIBRARY = any("gpu" in item.keywords for item in items)
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
