import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200) and the built library")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(autouse=True)
def _fresh_env_switches(request):
    """The library reads its POLESTAR_* switches once (at polestar_init / polestar_reload_env): after a GPU test
    that changed the environment, make the stand-alone kernel calls of later tests see the restored values.
    (Set up before `monkeypatch`, hence torn down after it has restored the environment.)"""
    yield
    if "gpu" in request.keywords:
        from paper_2607_14107_b200 import binding as Bd
        if Bd._lib is not None:
            Bd.polestar_reload_env()
