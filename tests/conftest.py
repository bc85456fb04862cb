import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")
    # the CUDA library and the oracle are built in-tree on first use (nvcc cross-compiles without a GPU)
    import __graft_entry__
    __graft_entry__.build()
