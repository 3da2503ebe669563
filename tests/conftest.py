import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
# some tests force a kernel variant through the library's developer switches; the library reads them only
# in processes started with this variable (it is looked at once, at the first call)
os.environ.setdefault("PRQ_DEV", "1")
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle (test infrastructure)."""
    from oracle import prq_oracle

    prq_oracle.build()
    return prq_oracle


@pytest.fixture(scope="session")
def prq():
    """The ctypes binding over libprq.so, built in-tree if needed."""
    from paper_2609_22106_b200 import binding, build

    build.build()
    binding.lib()
    return binding
