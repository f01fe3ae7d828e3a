import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
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
def _library_is_built():
    """The CUDA library is built in-tree and kept out of the history: a fresh checkout compiles it
    (nvcc, sm_100a; works without a GPU) before the first test needs it.  There is no other path to
    fall back to, so a failed build fails the session here."""
    from paper_2508_16201_b200 import specvlm
    if not os.path.exists(specvlm.LIB_PATH):
        from paper_2508_16201_b200 import build
        build.build()
    yield


@pytest.fixture(autouse=True)
def _poisoned_shared_memory(request):
    """Before every GPU test the SMs' shared memory is filled with NaN bit patterns: a kernel that
    reads a shared-memory word it never wrote then fails its parity check every time, instead of
    passing whenever the previous kernel happened to leave something harmless there."""
    if "gpu" in request.keywords:
        from paper_2508_16201_b200 import specvlm
        specvlm.debug_poison_shared_memory()
        specvlm.debug_fill_workspaces = True          # scratch buffers start as 0xff bytes, too
    yield
