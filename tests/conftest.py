import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


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


@pytest.fixture(scope="session", autouse=True)
def _native_code_is_built():
    """The C-ABI library and the oracle are compiled in-tree once per run if their sources are newer than the binaries
    (a no-op otherwise).  There is no other implementation to fall back to: a failed build fails the run."""
    from paper_2105_04246_b200 import build as hq_build
    import oracle
    hq_build.build()
    oracle.build()
