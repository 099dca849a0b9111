import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
for _p in (ROOT, os.path.join(ROOT, 'tests')):
    if _p not in sys.path:
        sys.path.insert(0, _p)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")
    # The C-ABI library and the C oracle are built in-tree; rebuild when sources are newer.
    from paper_2409_15104_b200 import build as pec_build
    from oracle import build as oracle_build
    pec_build.build()
    oracle_build.build()


@pytest.fixture(scope="session")
def pec():
    """The ctypes binding of the GPU library; GPU tests fail loudly when it is missing."""
    from paper_2409_15104_b200 import binding
    binding.load()
    return binding
