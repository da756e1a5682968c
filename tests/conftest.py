import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
# the mutation test runs the checker's pins against altered builds of the checker: a directory holding another
# `oracle` package takes precedence when named here
if os.environ.get("FCSIM_ORACLE_ROOT"):
    sys.path.insert(0, os.environ["FCSIM_ORACLE_ROOT"])


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    config.addinivalue_line("markers", "mutation: plants mistakes in copies of the CPU checker and expects its pins to fail")


def pytest_collection_modifyitems(config, items):
    # tests that need a GPU carry the marker explicitly; nothing is skipped silently here
    return


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
