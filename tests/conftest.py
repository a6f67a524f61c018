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


@pytest.fixture(autouse=True, scope="session")
def _debug_bounds_build():
    """With SHARPV_LIBRARY pointing at the range-checking build (libsharpv_debug.so, version 2xx) every call
    through the binding gets a status word, is followed by a synchronise, and fails the test if a kernel
    reported an index out of range.  This stands in for compute-sanitizer's memcheck on the kernels' own
    gather and scatter indices."""
    if not os.environ.get("SHARPV_LIBRARY"):
        yield
        return
    import torch
    from paper_2511_08003_b200 import binding as sv
    if not torch.cuda.is_available() or sv.lib().sharpv_version() < 200:
        yield
        return
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    plain = sv._call

    def checked(name, on, *args):
        args = list(args)
        mine = args[-2] is None and name not in ("sharpv_version",)
        if mine:
            args[-2] = word.data_ptr()
        rc = plain(name, on, *args)
        torch.cuda.synchronize()
        if mine:
            got = int(word.item())
            word.zero_()
            assert got != sv.Status.ERR_BOUNDS, f"{name}: a kernel reported an index out of range"
        return rc

    sv._call = checked
    yield
    sv._call = plain
