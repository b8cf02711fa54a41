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
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(params=[1, 2], ids=["warp_mma_attention", "tcgen05_attention"])
def attention_kind(request):
    """Plans made inside the test are laid out for the named attention kernel (the default leaves the
    choice to the planner's cost model)."""
    import paper_2511_07423_b200 as syn
    syn.debug_set_attention(request.param)
    yield request.param
    syn.debug_set_attention(0)
