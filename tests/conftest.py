import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, when no device is present."""
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


class _Tuning:
    """Sets KF_* dispatch switches for one test: the library reads its environment once, so
    every change is followed by kf_reload_tuning(); everything is undone, and reloaded, at
    teardown."""

    def __init__(self, monkeypatch):
        self._mp = monkeypatch

    def _reload(self):
        import paper_2605_30359_b200 as kf
        kf.kf_reload_tuning()

    def setenv(self, name, value):
        self._mp.setenv(name, value)
        self._reload()

    def delenv(self, name):
        self._mp.delenv(name, raising=False)
        self._reload()


@pytest.fixture
def tuning(monkeypatch):
    t = _Tuning(monkeypatch)
    yield t
    monkeypatch.undo()
    t._reload()
