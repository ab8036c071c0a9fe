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


def pytest_generate_tests(metafunc):
    """GPU tests that take `attention_path` run once per attention path of the library: 0 = warp-level
    MMAs (lane-owned tiles at every width), 1 = tensor memory (row tiles at 4 and 2 bit)."""
    if "attention_path" in metafunc.fixturenames:
        metafunc.parametrize("attention_path", [0, 1], ids=["warp_mma", "tensor_memory"])
