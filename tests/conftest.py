import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# Build the CUDA library (nvcc cross-compiles without a GPU) and the C oracle
# before any test module imports them.
sys.path.insert(0, os.path.join(ROOT, "paper_2310_10537_b200"))
import importlib.util  # noqa: E402

_spec = importlib.util.spec_from_file_location(
    "_mx_build", os.path.join(ROOT, "paper_2310_10537_b200", "build.py"))
_mx_build = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(_mx_build)
_mx_build.build()
sys.path.pop(0)

import oracle  # noqa: E402

oracle.build()


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
