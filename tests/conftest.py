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
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _error_log(request):
    """With LKV_ERR_LOG=<file>, append every test's measured max-relative errors to that file."""
    import helpers
    helpers.ERRORS.clear()
    yield
    path = os.environ.get("LKV_ERR_LOG")
    if path and helpers.ERRORS:
        with open(path, "a") as fh:
            fh.write(request.node.nodeid + " " + " ".join(f"{e:.3e}" for e in helpers.ERRORS) + "\n")


@pytest.fixture(autouse=True)
def _device_status_clean(request):
    """After every GPU test: no kernel of the library gave up a bounded wait on any workspace the binding handed out."""
    yield
    if "gpu" not in request.node.keywords:
        return
    from paper_2608_11231_b200 import binding as b
    for ws in list(b._ws_cache.values()):
        assert b.lkv_device_status(ws) == b.LKV_OK, "a device-side wait timed out during this test"
