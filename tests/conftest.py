import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle (compiled with gcc on first use)."""
    from oracle import gls_oracle

    gls_oracle.lib()
    return gls_oracle


@pytest.fixture(scope="session")
def gls():
    """The CUDA library binding; GPU tests fail loudly if it cannot be loaded."""
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2506_05632_b200 as pkg

    pkg.load()
    return pkg
