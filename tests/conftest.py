import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def lib():
    """The GPU library binding; GPU tests fail loudly if the extension or a device is missing."""
    import torch

    import paper_2104_04731_b200 as b2c

    b2c.load()
    assert torch.cuda.is_available(), "gpu-marked tests need a CUDA device"
    return b2c
