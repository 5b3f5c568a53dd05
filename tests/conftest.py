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
def _poison_outputs():
    """Outputs start from a sentinel: nothing passes on values left in recycled device memory."""
    try:
        import paper_2606_12370_b200.binding as binding
    except Exception:
        yield
        return
    old = binding.POISON_OUTPUTS
    binding.POISON_OUTPUTS = True
    yield
    binding.POISON_OUTPUTS = old
