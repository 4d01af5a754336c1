import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def basp():
    """The CUDA binding; building the library first if it is not there yet."""
    import __graft_entry__ as ge
    ge.build()
    from paper_2609_03151_b200 import binding
    return binding
