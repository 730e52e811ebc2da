import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--sweep-points", type=int, default=0,
                     help="run tests/test_gpu_sweep_full.py on this many seeded sweep points (0: skip it)")
    parser.addoption("--sweep-budget", type=float, default=1500.0, help="seconds for that run")
    parser.addoption("--sweep-out", default=None, help="JSON lines of that run, one per point")
    parser.addoption("--sweep-tile", default="off", choices=["off", "auto"],
                     help="let every plan of that run choose a tile basis")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def _have_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    if _have_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
