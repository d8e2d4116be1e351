import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")

_needs_cuda_library = False


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """The oracle's pins need only the oracle: the CUDA library is compiled when some other test is selected."""
    global _needs_cuda_library
    _needs_cuda_library = any(not os.path.basename(str(item.fspath)).startswith("test_oracle_") for item in items)


def golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


@pytest.fixture(scope="session", autouse=True)
def _built():
    """Compile the oracle's C core, and the CUDA library if a selected test uses it, once if they are missing."""
    import oracle
    oracle.build()
    if _needs_cuda_library:
        import __graft_entry__
        __graft_entry__.build()
