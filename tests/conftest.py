import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


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


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """The CUDA library is built in-tree before any test uses it (incremental: a no-op when it is up to date).
    If the build cannot run but a library is already there, the tests use that one; the binding itself raises
    when there is none."""
    try:
        from paper_2410_18035_b200 import build
        build.build()
    except Exception:
        from paper_2410_18035_b200.binding import LIB_PATH
        if not os.path.exists(LIB_PATH):
            raise
    yield
