import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")


@pytest.fixture(scope="session")
def batq():
    """The ctypes binding of the C-ABI library; GPU tests fail loudly if the
    library or the device is missing."""
    import torch
    from paper_2603_16590_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()
    return binding
