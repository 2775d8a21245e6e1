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
    from oracle import skim_oracle
    skim_oracle.build()
    return skim_oracle


@pytest.fixture(scope="session")
def skimlib():
    """The CUDA path: builds libskim.so if needed and returns the binding module."""
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2412_04180_b200 import build, skim
    build.build()
    skim.lib()
    return skim


@pytest.fixture()
def ctx(skimlib):
    c = skimlib.Skim(device=0)
    yield c
    c.close()
