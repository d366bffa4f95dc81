import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device in this process")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _bounds_report(request):
    """With UBT_LIB=checked (the range-checked debug build) fail a GPU test that indexed out of range."""
    yield
    if os.environ.get("UBT_LIB") != "checked" or "gpu" not in request.keywords:
        return
    import ctypes as C

    import torch

    import paper_2609_39972_b200 as u
    torch.cuda.synchronize()
    lib = u.load()
    for which, name in enumerate(("top-k", "tree", "verify")):
        out = (C.c_longlong * 4)()
        lib.ubt_debug_bounds_report(which, out)
        assert out[0] == 0, f"{name} kernels: index {out[2]} outside [0,{out[3]}) at site {out[1]}"
