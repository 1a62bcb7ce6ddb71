import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the library's kernels)")


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


@pytest.fixture(autouse=True)
def guard_bytes_checked_when_a_context_closes(request, monkeypatch):
    """Every GPU test that closes a context first has the library read back the guard bytes behind each of its
    workspaces (gn_debug_check_canaries): a kernel that wrote past the end of one fails the test that ran it."""
    if "gpu" not in request.keywords:
        yield
        return
    import paper_1802_00130_b200 as gn
    plain_close = gn.GnContext.close

    def close(self):
        if getattr(self, "_h", None):
            assert self.debug_check_canaries() > 0
        plain_close(self)

    monkeypatch.setattr(gn.GnContext, "close", close)
    yield
