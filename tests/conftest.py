import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _build_library_if_missing():
    """A clean checkout has no libgpd.so (built artefacts are not tracked): compile it once with nvcc,
    so that the suite can be run directly.  Nothing is built when the library is already there."""
    lib = os.path.join(ROOT, "paper_1811_10751_b200", "libgpd.so")
    if os.path.exists(lib):
        return
    import importlib.util
    spec = importlib.util.spec_from_file_location("_gpd_build", os.path.join(ROOT, "paper_1811_10751_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build(force=False)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (run with -m gpu on a B200)")
    _build_library_if_missing()
