import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--report-dir", default=None,
                     help="directory that receives the per-layer parity tables of the encoder tests "
                          "(error / allowed for every tensor of every layer); nothing is written without it")


@pytest.fixture(scope="session")
def report_dir(request):
    d = request.config.getoption("--report-dir")
    if d:
        os.makedirs(d, exist_ok=True)
    return d


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


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
