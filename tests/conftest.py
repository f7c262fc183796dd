import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped (not failed) on a machine without a device."""
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def path_switch(monkeypatch):
    """Set one of the library's DPCLIP_* path switches for the duration of a test.  The library reads them
    once, so it is told to re-read after the change and again after the variable has been restored."""
    import paper_2009_03106_b200 as pkg

    def set_switch(name, value):
        monkeypatch.setenv(name, value)
        pkg.dpclip_reload_path_switches()

    yield set_switch
    monkeypatch.undo()
    pkg.dpclip_reload_path_switches()
