import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def cuda_lib():
    """The CUDA library's Python binding; fails loudly if it cannot run on this machine."""
    import torch

    if not torch.cuda.is_available():
        pytest.fail("a test marked gpu ran on a box without a CUDA device")
    import paper_2502_07861_b200 as bk

    bk.load()
    return bk
