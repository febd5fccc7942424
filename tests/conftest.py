import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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
def kvm_lib():
    """The CUDA library, built in-tree when stale.  Tests that only need its host side are skipped on a
    machine that has neither nvcc nor a prebuilt libkvm.so, instead of failing there."""
    import shutil
    from paper_2407_08454_b200 import binding, build
    try:
        if shutil.which(os.environ.get("NVCC", "nvcc")):
            build.build()
        return binding.lib()
    except (FileNotFoundError, OSError, RuntimeError) as exc:
        pytest.skip(f"libkvm.so cannot be built or loaded here: {exc}")
