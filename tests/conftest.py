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
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _canaries_after_every_gpu_test(request):
    """Every buffer the tests hand to the library through runtime.PathAttention (KV pool, workspace,
    outputs it allocates) sits between two canary bands; after each GPU test the bands of every
    handle still alive are checked (closed handles were checked when they closed)."""
    yield
    if "gpu" in request.keywords:
        from paper_2605_22566_b200 import runtime
        runtime.verify_all_guards()
