import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def lib():
    """The ctypes binding with the C-ABI library loaded (built on demand)."""
    from paper_2609_33645_b200 import build
    build.build()
    from paper_2609_33645_b200 import binding
    binding.load()
    return binding
