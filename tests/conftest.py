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
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def options():
    """Sets tuning options of the library for one test (``options(option_id, value)``) and puts the
    previous values back afterwards."""
    from paper_2603_12617_b200 import binding
    saved = {}

    def set_option(option_id, value):
        saved.setdefault(option_id, binding.sd_get_option(option_id))
        binding.sd_set_option(option_id, value)

    yield set_option
    for option_id, value in saved.items():
        binding.sd_set_option(option_id, value)
