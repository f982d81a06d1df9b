import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu")


def pytest_sessionstart(session):
    """Build the shared library when it is missing or older than its sources (nvcc cross-compiles without a GPU)."""
    try:
        from paper_2506_09316_b200 import build
        build.build()
    except Exception as e:  # the tests that need the library then fail loudly on import
        print(f"[conftest] could not build libdsla.so: {e}", file=sys.stderr)


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(params=["tensor", "pair"])
def tc_impl(request):
    """Both tensor-core prefill variants: both states in one CTA / one state per CTA of a two-CTA cluster."""
    return request.param
