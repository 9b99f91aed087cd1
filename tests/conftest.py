import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200 with -m gpu)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import kvpo
    kvpo.build()
    return kvpo


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """The CUDA library is built in-tree (nvcc, sm_100a) if it is missing or older than its sources."""
    from paper_2508_13231_b200 import build
    build.build_library()


@pytest.fixture
def hooks():
    """Sets the library's test switches (kvp_set_test_hooks) for one test and clears them afterwards.
    Call it with keyword arguments; every call replaces the previous setting."""
    from paper_2508_13231_b200 import kvp
    state = {}

    def set_hooks(**kw):
        state.update(kw)
        kvp.set_test_hooks(**state)

    yield set_hooks
    kvp.set_test_hooks()
