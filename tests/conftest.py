import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_sessionstart(session):
    # A child run of the suite may ask for one attention kernel (tests/test_gpu_attention_fallback.py).
    which = os.environ.get("CATS_TEST_ATTENTION_KERNEL")
    if which is not None:
        import torch
        if torch.cuda.is_available():
            from paper_2605_11186_b200 import binding
            binding.attention_kernel(int(which))


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
