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
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(params=["streaming", "ring", "cluster"])
def kernel_path(request):
    """Runs a GPU test once per kernel set (the ring set falls back to streaming, the one-launch
    cluster form to the automatic choice, for shapes they do not take, so every parametrisation is
    always valid)."""
    from paper_2411_00853_b200 import binding
    binding.set_path({"streaming": binding.PATH_STREAMING, "ring": binding.PATH_RING,
                      "cluster": binding.PATH_CLUSTER}[request.param])
    yield request.param
    binding.set_path(binding.PATH_AUTO)
