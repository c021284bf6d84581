import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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
def _built_libraries():
    """The CUDA library (nvcc cross-compiles without a GPU) and the C oracle are built in-tree before any
    test runs; a failed build fails the session instead of letting tests look for a missing library."""
    from paper_2604_09244_b200 import build
    import oracle
    build.build_library()
    oracle.build()


def pytest_terminal_summary(terminalreporter):
    """How many parity checks sat on a threshold (and were judged by the rules on the GPU's own indicators)."""
    try:
        import parity_util
    except Exception:
        return
    if parity_util.LENIENT:
        terminalreporter.write_line(f"parity checks on a threshold: {len(parity_util.LENIENT)} "
                                    f"(first: {parity_util.LENIENT[0]})")
