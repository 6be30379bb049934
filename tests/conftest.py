import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    config.addinivalue_line("markers", "slow: long-running pin, opt in with SPS_SLOW=1")


def pytest_collection_modifyitems(config, items):
    if os.environ.get("SPS_SLOW") == "1":
        return
    skip = pytest.mark.skip(reason="set SPS_SLOW=1 to run")
    for it in items:
        if "slow" in it.keywords:
            it.add_marker(skip)
