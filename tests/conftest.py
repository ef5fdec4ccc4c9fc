import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def ciar_lib():
    """The built C-ABI library, compiled here if it is missing or older than its sources."""
    from paper_2603_25463_b200 import build as _build
    _build.build_library()
    from paper_2603_25463_b200 import ciar
    return ciar
