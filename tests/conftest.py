import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_sessionstart(session):
    """A fresh checkout has no compiled library yet; the package refuses to import without it.  Build it (nvcc
    cross-compiles without a GPU) before any test module is imported.  The build script is loaded by path because
    importing the package is exactly what needs the library."""
    import importlib.util
    import shutil
    path = os.path.join(ROOT, "paper_2607_16784_b200", "build.py")
    spec = importlib.util.spec_from_file_location("_roomie_build", path)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    if os.path.exists(os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")) or shutil.which("nvcc"):
        mod.build()                                  # no-op when the library is newer than its sources


@pytest.fixture(scope="session")
def oracle():
    import oracle as o
    o.build()
    return o
