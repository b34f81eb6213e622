import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    # Make sure the shared library matches the sources (a no-op when it is up to date).  The
    # tests never fall back to anything else: without nvcc and without a built library they fail.
    try:
        from paper_1801_04928_b200 import build as lfbuild
        lfbuild.build()
    except Exception as exc:  # pragma: no cover
        sys.stderr.write(f"[conftest] could not (re)build libleapfrog.so: {exc}\n")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
