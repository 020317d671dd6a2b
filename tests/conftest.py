import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def cuda_lib():
    """The loaded C-ABI binding; GPU tests fail loudly if the CUDA library is missing."""
    import torch

    assert torch.cuda.is_available(), "gpu-marked test run without a CUDA device"
    from paper_2507_19906_b200 import binding

    binding.load()  # raises if the shared library is not built
    return binding
