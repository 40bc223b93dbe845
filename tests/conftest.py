import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device and the built CUDA library")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """The CUDA library, built in-tree from the sources if it is missing or older than them (a no-op otherwise).
    There is nothing else for the tests to run: a failed build fails the session."""
    from paper_2310_14423_b200 import build as qsr_build
    qsr_build.build()
