import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import oracle as o
    o.lib()
    return o


@pytest.fixture(scope="session", autouse=True)
def _preloaded_helper_kernels():
    """GPU runs: load the helper kernels before any test scripts a producer behind an already waiting reducer."""
    try:
        import torch
        if torch.cuda.is_available():
            from paper_2607_08973_b200 import binding as sf
            sf.sifar_workload_preload()
    except ImportError:
        pass
    yield
