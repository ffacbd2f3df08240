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


@pytest.fixture
def verify_schedule(request):
    """Runs a verification test once per schedule of seq_tree_verify (node-parallel, walk)."""
    from tests import gpu_util as G

    G.SCHEDULE = request.param
    yield request.param
    G.SCHEDULE = "auto"


def pytest_generate_tests(metafunc):
    name = metafunc.function.__name__
    if ((metafunc.module.__name__.split(".")[-1] in ("test_gpu_parity", "test_gpu_parity_full") and name.startswith("test_verify")
         or metafunc.module.__name__.split(".")[-1] == "test_gpu_greedy" and "verify_schedule" in metafunc.fixturenames)
            and "every_node_hook" not in name):
        if "verify_schedule" not in metafunc.fixturenames:
            metafunc.fixturenames.append("verify_schedule")
        metafunc.parametrize("verify_schedule", ["nodes", "walk"], indirect=True)
