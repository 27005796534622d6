import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_sessionstart(session):
    # a checkout without the built library (it is not under version control): compile it once, in-tree
    lib = os.path.join(ROOT, "paper_2603_04135_b200", "libdppo.so")
    if not os.path.exists(lib):
        from paper_2603_04135_b200 import build
        build.build_library()


def pytest_collection_modifyitems(config, items):
    # GPU tests are skipped (not failed) when collected on a box without a device and without -m gpu
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
