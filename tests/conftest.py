import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _ensure_library():
    """Build libet.so in-tree if it is missing or older than its sources (the build script compares
    modification times itself and returns at once when the library is fresh; it is run as a script
    because importing the package needs the library)."""
    import subprocess
    script = os.path.join(ROOT, "paper_2312_14227_b200", "build.py")
    subprocess.run([sys.executable, script], check=True, capture_output=True)


_ensure_library()


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


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
