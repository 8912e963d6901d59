import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a B200 and the built CUDA library")


@pytest.fixture(scope="session")
def orc():
    from oracle import mp_oracle
    mp_oracle.build()
    return mp_oracle


@pytest.fixture(scope="session")
def mp():
    """The Python binding of the CUDA library; GPU tests only."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1805_10387_b200 import mp as binding
    binding.lib()
    return binding
