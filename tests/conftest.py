import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built CUDA library")


def pytest_collection_modifyitems(config, items):
    # Files named test_zz_* are collected last so that a run that stops at the first failure
    # has already exercised everything else.
    items.sort(key=lambda it: (1 if os.path.basename(str(it.fspath)).startswith("test_zz_") else 0))


@pytest.fixture(scope="session")
def cuda_device():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


@pytest.fixture(autouse=True)
def _device_status_stays_clear(request):
    """Every GPU test ends with a clear device status word: no bounded wait ran out and (checked build) no bounds
    predicate failed in any kernel the test launched.  Tests that provoke a status read it themselves, which clears it."""
    yield
    if request.node.get_closest_marker("gpu") is None:
        return
    import torch
    if not torch.cuda.is_available():
        return
    import paper_2608_03537_b200 as cf
    assert cf.last_device_status() == cf.OK, "a kernel launched by this test left a device status behind"
