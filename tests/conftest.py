import os
import sys

# the tests steer kernel variants through the library's experiment knobs, which it only reads
# in a process started with this variable set
os.environ.setdefault("QKNORM_DEBUG_ENV", "1")

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


@pytest.fixture(scope="session")
def libqknorm():
    """Builds (if stale) and loads the CUDA library; every test that touches the C ABI uses this."""
    from paper_2608_09160_b200 import binding, build
    build.build()
    return binding.load()
