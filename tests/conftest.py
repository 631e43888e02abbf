import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_sessionstart(session):
    """The tests run against the in-tree library: bring it up to date with the sources once per
    session (a no-op when it is fresh).  If the compiler is not available the existing file is used."""
    try:
        from paper_2602_12305_b200 import build
        build.build_library()
    except Exception as e:                      # noqa: BLE001 -- reported, then the tests decide
        print(f"[conftest] could not rebuild the library ({e}); using the file on disk")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
