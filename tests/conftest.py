import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


# The CUDA library is built in-tree; build it here if this checkout has none yet
# (loading build.py by path, since importing the package already needs the library).
try:
    import importlib.util as _ilu
    _spec = _ilu.spec_from_file_location("_zoa_build", os.path.join(ROOT, "paper_2202_06009_b200", "build.py"))
    _mod = _ilu.module_from_spec(_spec)
    _spec.loader.exec_module(_mod)
    _mod.build()
except Exception as exc:  # nvcc missing: the tests that need the library will say so
    print(f"[conftest] could not build libzoa.so: {exc}")
