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
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device in this process")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def debug_switch():
    """Turns one of the library's test switches (nq_debug_set) on for the rest of a test and off again afterwards."""
    import paper_2506_17870_b200 as nq
    used = []

    def on(which):
        nq.nq_debug_set(which, True)
        used.append(which)

    yield on
    for which in used:
        nq.nq_debug_set(which, False)
