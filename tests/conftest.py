import os
import sys
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_sessionstart(session):
    # Build the CUDA library and the C oracle in-tree if they are missing or older than their sources, so that a
    # fresh checkout can run the suite directly.  A failure here is left for the tests that need the library to report.
    try:
        from paper_2109_12191_b200 import build as libbuild
        libbuild.build()
        import oracle
        oracle.build()
    except Exception as exc:  # noqa: BLE001
        print(f"[conftest] in-tree build failed: {exc}")


def pytest_collection_modifyitems(config, items):
    # GPU tests can only run where a device exists; elsewhere they are skipped, never emulated.
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
