import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def repo_root():
    return ROOT


@pytest.fixture(scope="session")
def rfast_lib():
    """The built shared library (compiled on first use; nvcc cross-compiles without a GPU)."""
    from paper_2307_11617_b200.build import build
    build()
    from paper_2307_11617_b200 import binding
    return binding.lib()


def has_cuda():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False
