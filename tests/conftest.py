import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")
    config.addinivalue_line("markers", "slow: long-running full-size parity case")


def pytest_collection_modifyitems(config, items):
    # files named test_zz_* are collected last already (alphabetical); keep that order stable
    items.sort(key=lambda it: (os.path.basename(str(it.fspath)).startswith("test_zz_"),))
