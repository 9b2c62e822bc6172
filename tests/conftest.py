import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
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


@pytest.fixture(scope="session", autouse=True)
def _linear_algo_override():
    """AKVS_TEST_LINEAR_ALGO=1 runs the bf16 pipeline tests on the CUDA-core linear kernels
    (a cross-check of the tensor-core ones); the default is the product configuration."""
    algo = os.environ.get("AKVS_TEST_LINEAR_ALGO")
    if algo is not None:
        import paper_2607_21604_b200 as a
        a.lib.akvs_debug_set_linear_algo(int(algo))
    yield
