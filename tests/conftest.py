import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_addoption(parser):
    parser.addoption("--checked-build", action="store_true", default=False,
                     help="run the GPU tests through the checked build of the library: index tests compiled into the kernels, "
                          "an index outside its array fails the test through the status word")


@pytest.fixture(scope="session", autouse=True)
def _library_form(request):
    if not request.config.getoption("--checked-build"):
        yield
        return
    from paper_2603_06626_b200 import binding
    with binding.checked_build():
        yield


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
