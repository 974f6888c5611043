import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_addoption(parser):
    parser.addoption("--checked-library", action="store_true",
                     help="run against libegeria_checked.so (index checks inside the kernels)")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


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
def _built_library():
    """The CUDA library is built in-tree (nvcc cross-compiles without a GPU)."""
    from paper_2201_06227_b200 import build
    build.build()


@pytest.fixture(scope="session", autouse=True)
def _which_library(request, _built_library):
    """With --checked-library every test of the session talks to the checked build."""
    if request.config.getoption("--checked-library"):
        from paper_2201_06227_b200 import binding
        binding.use_checked_library(True)
        assert binding.lib().egeria_build_is_checked() == 1
