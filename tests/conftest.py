import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a B200 (sm_100a) GPU; calls the CUDA library through the C ABI")


def pytest_collection_modifyitems(config, items):
    # keep alphabetical file order (the no-GPU default), so files named test_zz_* run last
    items.sort(key=lambda it: (os.path.basename(str(it.fspath)),))


@pytest.fixture(scope="session")
def cuda_device():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("a test marked gpu ran without a CUDA device")
    major, minor = torch.cuda.get_device_capability(0)
    if major != 10:
        pytest.fail(f"these kernels are sm_100a only; found sm_{major}{minor}")
    return torch.device("cuda:0")
