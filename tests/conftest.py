import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import heinsen_oracle
    heinsen_oracle.build()
    return heinsen_oracle

TESTS = os.path.dirname(os.path.abspath(__file__))
if TESTS not in sys.path:
    sys.path.insert(0, TESTS)


@pytest.fixture(scope="session")
def hs():
    """The Python binding over the C ABI, with the library built; GPU tests only."""
    import torch
    from paper_2311_06281_b200 import build_ext, heinsen_scan
    build_ext.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    heinsen_scan.lib()
    return heinsen_scan


@pytest.fixture(autouse=True)
def _reset_path(request):
    yield
    if "hs" in request.fixturenames:
        from paper_2311_06281_b200 import heinsen_scan
        heinsen_scan.set_path(heinsen_scan.PATH_AUTO)
        heinsen_scan.debug_config(0, -1)
