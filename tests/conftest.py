import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def nm():
    """The CUDA library binding; GPU tests fail loudly if it cannot load or no device is present."""
    import torch
    import paper_2305_14405_b200 as pkg
    assert torch.cuda.is_available(), "GPU test selected but no CUDA device is visible"
    pkg.load()
    return pkg
