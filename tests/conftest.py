import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device in this process")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """The GPU tests call the in-tree CUDA library: compile it first if it is missing or older than its
    sources (needs nvcc; without it the tests that need the library fail loudly, there is no fallback)."""
    try:
        from paper_2104_08378_b200 import build
        if build.needs_build():
            build.build_library()
    except Exception as e:  # noqa: BLE001 - reported by the tests that need the library
        print(f"could not build libsp24.so: {e}", file=sys.stderr)
    yield


@pytest.fixture
def force_tile():
    """force_tile("2x224x2") makes every GEMM call of the test use that tile shape; the automatic
    choice is restored afterwards."""
    from paper_2104_08378_b200 import binding
    yield binding.set_tile_override
    binding.set_tile_override(None)
