import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_libraries():
    """Builds what the tests load if it is missing or older than its sources: the CUDA library
    (nvcc cross-compiles without a GPU) and the C checker.  The package itself never builds on
    import and fails loudly when its library is absent."""
    import shutil
    if shutil.which("nvcc"):
        from paper_2603_01501_b200 import build as gbuild
        gbuild.build()
    from oracle import gac_oracle
    gac_oracle.build()
    yield
