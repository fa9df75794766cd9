import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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
def _default_library_options():
    """Every test starts from, and leaves behind, the library's default options."""
    yield
    try:
        from paper_2202_00441_b200 import binding
    except Exception:  # pragma: no cover
        return
    if binding._lib is not None:
        for opt, default in ((0, 0), (1, 0), (2, 0), (3, 0), (4, 1), (5, 0), (6, 0)):
            binding._lib.fewbit_set_option(opt, default)
