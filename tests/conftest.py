import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")
    # a fresh checkout has no library yet (it is built in-tree, not committed): build it once where nvcc exists
    lib = os.path.join(ROOT, "paper_2403_00176_b200", "libsod2.so")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(lib) and os.path.exists(nvcc):
        from paper_2403_00176_b200 import build as _build
        _build.build()


def pytest_collection_modifyitems(config, items):
    # tests in files named test_zz_* run after everything else
    items.sort(key=lambda it: (os.path.basename(str(it.fspath)).startswith("test_zz_"),))
