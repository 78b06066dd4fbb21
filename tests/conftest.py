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


@pytest.fixture(scope="session", autouse=True)
def _library_is_the_requested_build():
    """A run that was asked to use the bounds-checked library (EG_EXPECT_DEBUG) must not fall back
    silently to the ordinary one."""
    if os.environ.get("EG_EXPECT_DEBUG"):
        from paper_2103_07454_b200 import binding
        assert binding.load_library().eg_debug_build() == 1, "EG_LIBRARY does not name the bounds-checked build"
    yield
