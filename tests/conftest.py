import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def tuning():
    """Apply overrides of the library's launch planner for one test: tuning(splits=3, kernel=2). Reset afterwards."""
    from paper_2508_02558_b200 import binding as B
    B.tuning_reset()

    def apply(**kw):
        for name, value in kw.items():
            B.tuning_set(name, value)
    yield apply
    B.tuning_reset()
