"""Shared pytest configuration: the ``gpu`` marker and import paths."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _build_library_if_missing():
    """The package refuses to import without its CUDA library (no fallback path), and the built file is not
    tracked: compile it once per checkout by running the build script, which needs nvcc but no GPU."""
    import importlib.util

    spec = importlib.util.spec_from_file_location("_pd_build_script", os.path.join(ROOT, "paper_2609_35158_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build_library()  # no-op when the library is newer than its sources


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    _build_library_if_missing()


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
