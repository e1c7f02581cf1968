"""Shared pytest configuration: the `gpu` marker, import path, and in-tree builds."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # The C-ABI library and the oracle are built in-tree; make sure both exist before collection.
    import glob
    import oracle
    oracle.build()
    if glob.glob(os.path.join(ROOT, "paper_2607_28150_b200", "csrc", "*.cu")):
        import __graft_entry__ as entry
        entry.build(quiet=True)


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
