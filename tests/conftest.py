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
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def guarded_buffers():
    """Every Actor of the test-suite gets guard bytes around its ring, state and work buffers (the stand-in for a
    memory checker); they are verified when the actor is destroyed."""
    from paper_2205_05248_b200 import binding
    old = binding.GUARD_BYTES
    binding.GUARD_BYTES = 4096
    yield
    binding.GUARD_BYTES = old
