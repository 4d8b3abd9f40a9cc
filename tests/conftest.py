import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


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
def _library_switches_back_to_default():
    """Process-wide switches of the library a test may have flipped are put back after every test."""
    yield
    try:
        import paper_2603_13420_b200 as pskv
        pskv.pskv_set_multi_form("auto")
        pskv.pskv_enable_cta_pairs(False)
    except Exception:  # library not built: nothing to reset
        pass


@pytest.fixture(scope="session", autouse=True)
def _built_libraries():
    """Compile the CUDA library and the C oracle once per session if their sources changed."""
    from paper_2603_13420_b200 import build as pskv_build
    import oracle

    pskv_build.build()
    oracle.build()
