import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")


@pytest.fixture(scope="session")
def tb():
    """The Python binding of the CUDA library (built on demand where nvcc is present)."""
    from paper_2608_21343_b200 import build as tb_build
    tb_build.ensure_built()
    from paper_2608_21343_b200 import binding
    return binding
