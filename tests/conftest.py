import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session", autouse=True)
def _oracle_threads():
    # The oracle's loops over independent outputs may use every host core; results do
    # not depend on the thread count.
    from oracle import binding
    binding.set_threads(os.cpu_count() or 1)
    yield
