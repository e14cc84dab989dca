import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")
    # the CUDA library is built in-tree; build it if it is missing or older than its source (nvcc needs no GPU)
    try:
        from paper_2502_04677_b200 import build
        build.build()
    except Exception as e:      # the tests that need the library will say so themselves
        print("libklpm.so could not be built: %s" % e)


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
