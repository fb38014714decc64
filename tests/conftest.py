import os

os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")  # one hardware queue per scheduler stream; read when the CUDA context is created
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
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture
def conv_pair_tiles(monkeypatch):
    """Handles created in this test run wide convolution layers as SM-pair tiles (off by default: a
    handle keeps to one kind of tensor-memory allocation; the environment variable is read at lp_create)."""
    monkeypatch.setenv("LP_CONV_PAIR", "1")
