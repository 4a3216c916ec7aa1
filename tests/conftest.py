import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


def read_printed_values():
    """name -> float, from tests/golden/paper_printed_values.txt."""
    out = {}
    with open(os.path.join(GOLDEN, "paper_printed_values.txt")) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


@pytest.fixture(scope="session")
def printed():
    return read_printed_values()


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """On a GPU machine make sure the in-tree CUDA library exists and is current before any GPU test loads it
    (the library is a build product and is not kept in version control)."""
    try:
        import torch
        if torch.cuda.is_available():
            from paper_2609_02846_b200.build import build_library
            build_library()
    except ImportError:
        pass
    yield
