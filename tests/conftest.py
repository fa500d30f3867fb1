import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the C-ABI library on it)")


@pytest.fixture(scope="session")
def libssn():
    """The C-ABI library through its Python binding; built in-tree on first use."""
    import __graft_entry__ as entry

    entry.build()
    from paper_2607_13332_b200 import binding

    return binding
