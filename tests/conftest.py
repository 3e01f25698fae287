import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _launch_mode():
    """ZQFP_TEST_EXCLUSIVE_DEVICE=1 runs the whole suite with the plain launches of zq_set_exclusive_device(1)
    (the test process has the GPU to itself); the default is the library's default, cooperative launches."""
    if os.environ.get("ZQFP_TEST_EXCLUSIVE_DEVICE") == "1":
        from paper_2307_09782_b200 import binding
        binding.set_exclusive_device(True)
    yield
