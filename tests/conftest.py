import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def lib():
    """The C-ABI library through its Python binding; built on demand if missing."""
    from paper_2606_03077_b200 import build as _build

    _build.build_library(verbose=False)
    from paper_2606_03077_b200 import binding

    return binding
