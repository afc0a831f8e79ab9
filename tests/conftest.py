import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    config.addinivalue_line("markers", "slow: full-size case that takes minutes")


def pytest_sessionstart(session):
    """Make sure the CUDA library exists before any test imports the package (the package
    refuses to import without it).  nvcc cross-compiles, so this also works without a GPU."""
    import importlib.util
    path = os.path.join(ROOT, "paper_1709_09393_b200", "build.py")
    spec = importlib.util.spec_from_file_location("_slimdp_cuda_build", path)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build()
