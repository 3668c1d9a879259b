import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")
    # the tests call the in-tree CUDA library through its C ABI: build it (nvcc, no GPU needed) when it is missing
    # or older than its sources, so that a fresh checkout can run the suite directly
    try:
        from paper_2509_22323_b200 import build as cuda_build
        cuda_build.build()
    except Exception as exc:  # pragma: no cover - reported by the tests that need the library
        print(f"conftest: could not build librapid3.so: {exc}")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
