import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def golden_lines(name):
    """Non-comment, non-empty lines of a golden fixture, split into fields."""
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.lstrip().startswith("#")]


@pytest.fixture(scope="session")
def lib():
    """The C-ABI library through its Python binding (built in-tree on first use)."""
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_15141_b200 import binding
    return binding
