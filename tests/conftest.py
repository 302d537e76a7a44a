import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, where no device exists."""
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_libraries():
    """Compile the CUDA libraries and the C oracle if they are missing or older than their sources
    (nvcc and gcc need no GPU), so that a fresh checkout can run either half of the suite."""
    from paper_2509_07506_b200 import build as astra_build
    astra_build.ensure_built()
    astra_build.ensure_built(ablation=True)
    import oracle
    oracle.build()
