import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_sessionstart(session):
    """The kernels of the seeded random test programs are not part of the product library: they live in a
    shared object of their own, built from tests/programs/ and loaded into the registry here."""
    from paper_2407_13585_b200 import binding, build
    if not os.path.exists(build.TEST_LIB):
        build.build_test_kernels()
    binding.load_kernel_library(build.TEST_LIB)


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
