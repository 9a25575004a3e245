import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (parity tests through the C ABI)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as orc

    orc.build()
    return orc


@pytest.fixture(scope="session")
def tfjsb():
    """The CUDA library's Python binding with a live context; GPU tests only."""
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_1901_05350_b200 as pkg

    return pkg


@pytest.fixture(scope="session")
def ctx(tfjsb):
    c = tfjsb.Context(0)
    yield c
    c.check_device_status()
    c.close()
