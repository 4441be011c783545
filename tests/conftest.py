import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(autouse=True)
def _side_stream(request):
    """GPU tests run on a non-default CUDA stream: the library captures its launch sequences
    into CUDA graphs, which the legacy default stream does not allow."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    import torch
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        yield
    torch.cuda.synchronize()
