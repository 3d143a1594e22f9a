import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


def pytest_sessionstart(session):
    """The shared library is a build artefact (not in version control): compile it when it is missing or older than
    its sources, so that neither the CPU nor the GPU suite depends on an earlier build step."""
    try:
        from paper_2302_06058_b200 import build
        build.build()
        build.build(debug=True)
    except Exception as exc:                                 # the tests that need the library will say so themselves
        sys.stderr.write(f"[conftest] building libbimask.so failed: {exc}\n")
