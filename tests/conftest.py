import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


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


@pytest.fixture(scope="session", autouse=True)
def _oracle_library():
    """Build the C oracle once per session if it is missing or stale (gcc only: the oracle's pins
    must run on a machine that has no CUDA toolkit)."""
    import oracle
    oracle.build()


@pytest.fixture(scope="session")
def cuda_library():
    """The CUDA library, built with nvcc if missing or stale; tests that need it are skipped,
    with the reason, where it can neither be found nor compiled."""
    import shutil
    from paper_2405_12528_b200 import build as builder
    try:
        return builder.build()
    except Exception as exc:                                  # no nvcc, failed compile
        if os.path.exists(builder.LIB) or shutil.which(os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")):
            raise
        pytest.skip(f"libsirllm.so is not built and nvcc is missing: {exc}")


@pytest.fixture(scope="session", autouse=True)
def _cuda_library_for_gpu_runs(request):
    """A run that collected GPU tests on a machine with a GPU builds the CUDA library up front."""
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu and any("gpu" in item.keywords for item in request.session.items):
        request.getfixturevalue("cuda_library")
