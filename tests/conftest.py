import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped (not failed) on a box without a CUDA device."""
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


@pytest.fixture(params=[0, 1], ids=["gelu-table", "gelu-computed"])
def gelu_mode(request):
    """Runs a test with FFN1's i-GELU looked up in the layer's table and computed per element."""
    from gpu_util import ctx
    c = ctx()
    c.ibert_set_gelu_table(request.param)
    yield request.param
    c.ibert_set_gelu_table(0)


@pytest.fixture(params=[0, 1, 2], ids=["inner-transposed", "inner-rows", "inner-transposed-any-size"])
def qkv_layout(request):
    """Runs a test with the layer's internal tensors (Q | K | V, the FFN1 result) transposed where shapes
    allow and sizes make it pay, in rows, and transposed wherever shapes allow."""
    from gpu_util import ctx
    c = ctx()
    c.ibert_set_qkv_layout(request.param)
    yield request.param
    c.ibert_set_qkv_layout(0)
