import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(params=[1, 2], ids=["one_tile_items", "two_tile_items"])
def both_window_kernels(request, monkeypatch):
    """The softmax window has two kernels, picked per launch from the number of work items: window_tc (two
    query tiles per item) and window_tc1 (one).  Small test shapes would all land on the second; this fixture
    runs a test once with each by setting rehyat_config.window_tiles for every context the test creates."""
    from paper_2601_04342_b200 import binding
    monkeypatch.setitem(binding.TUNING_DEFAULTS, "window_tiles", request.param)
    return request.param
