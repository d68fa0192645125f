import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--ngc-library", default=None,
                     help="run the GPU tests against another build of the CUDA library, for instance "
                          "paper_2604_18002_b200/libngc_b200_debug.so (the bounds-checking build)")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session", autouse=True)
def _ngc_library(request):
    """With --ngc-library every call of the binding goes to that build for the whole session."""
    path = request.config.getoption("--ngc-library")
    if not path:
        yield
        return
    from paper_2604_18002_b200 import binding
    with binding.use_library(os.path.abspath(path)):
        yield


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)
