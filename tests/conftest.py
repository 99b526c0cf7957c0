import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def repo_root():
    return ROOT


@pytest.fixture(scope="session", autouse=True)
def library_is_built():
    """Every test file talks to the in-tree shared library: build it once if it is missing or stale.  When the
    build cannot run (no compiler on this machine) an existing library is used as it is; with neither, the
    binding's own loud failure is what the tests report."""
    from paper_2512_12928_b200 import build as ps_build
    try:
        ps_build.build()
    except Exception:
        if not os.path.exists(ps_build.LIB_PATH):
            raise
