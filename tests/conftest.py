import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_runtest_setup(item):
    # a GPU-marked test that was selected on a box without a device fails loudly instead of
    # passing on some fallback or being skipped silently (deselect with -m "not gpu")
    if "gpu" in item.keywords:
        import torch
        if not torch.cuda.is_available():
            pytest.fail("this test needs a CUDA device; deselect it with -m \"not gpu\"", pytrace=False)
