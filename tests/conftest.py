import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); deselected on CPU-only runs")


def pytest_collection_modifyitems(config, items):
    # Files named test_zz_* run last so that a stop-at-first-failure run has covered everything else.
    items.sort(key=lambda it: (os.path.basename(str(it.fspath)).startswith("test_zz_"),))


@pytest.fixture(scope="session")
def repo_root():
    return ROOT


@pytest.fixture(scope="session", autouse=True)
def built_library():
    """The shared library is built in-tree once per session if it is missing or older than its sources
    (nvcc cross-compiles without a GPU); a failing build fails the tests that need it, loudly."""
    from paper_2505_21036_b200 import build
    return build.build()
