import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")
    config.addinivalue_line("markers", "slow: takes many minutes (full decode lengths); runs only with DYNAKV_RUN_SLOW=1")


def pytest_sessionstart(session):
    # a run that asks for the bounds-checked library must really get it
    if os.environ.get("DYNAKV_LIBRARY") == "checked":
        import paper_2511_07427_b200 as P
        assert P.load_library().dynakv_checked_build() == 1, "DYNAKV_LIBRARY=checked, but the loaded library has no index tests"


def pytest_collection_modifyitems(config, items):
    if os.environ.get("DYNAKV_RUN_SLOW") == "1":
        return
    skip = pytest.mark.skip(reason="slow: set DYNAKV_RUN_SLOW=1 to run the full decode lengths")
    for item in items:
        if "slow" in item.keywords:
            item.add_marker(skip)
