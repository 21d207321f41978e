import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the kernels through the C-ABI)")
    config.addinivalue_line("markers", "slow: long-running parity case")


def pytest_collection_modifyitems(config, items):
    # A test file whose name starts with test_zz_ is meant to run after every other file.
    items.sort(key=lambda it: (os.path.basename(str(it.fspath)).startswith("test_zz_"),))


@pytest.fixture(scope="session")
def has_gpu():
    import torch
    return torch.cuda.is_available()


@pytest.fixture(params=["auto", "scan"])
def router(request):
    """Runs a routing test once with the library's choice of kernel and once with the scanning kernel."""
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200.state import DeviceState
    old = DeviceState.default_router
    DeviceState.default_router = {"auto": B.ROUTE_AUTO, "scan": B.ROUTE_SCAN}[request.param]
    yield request.param
    DeviceState.default_router = old
