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
    """Fail a GPU test during which a device-side wait gave up or (UBT_LIB=checked) an index was out of range."""
    yield
    if "gpu" not in request.keywords:
        return
    import ctypes as C

    import torch

    import paper_2609_39972_b200 as u
    if not torch.cuda.is_available():
        return
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0, "a bounded device-side wait gave up"
    if os.environ.get("UBT_LIB") != "checked":
        return
    lib = u.load()
    for which, name in enumerate(("top-k", "tree", "verify")):
        out = (C.c_longlong * 4)()
        lib.ubt_debug_bounds_report(which, out)
        assert out[0] == 0, f"{name} kernels: index {out[2]} outside [0,{out[3]}) at site {out[1]}"
