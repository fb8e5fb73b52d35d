import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (parity tests against the CPU oracle)")


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


@pytest.fixture(autouse=True)
def _memory_safety(request):
    """After every GPU test: no buffer of a live harness session has been written outside its bounds (guard bytes
    around every device buffer), and, when the checked build of the library is loaded (BAOC_CHECKED=1), none of its
    kernels has recorded a violation."""
    yield
    if "gpu" not in request.keywords:
        return
    B = sys.modules.get("paper_2605_04711_b200.binding")
    H = sys.modules.get("paper_2605_04711_b200.harness")
    if B is not None:
        status = B.check_status()
        assert status["code"] == 0, status
    if H is not None and H.LIVE_SESSIONS:
        for sess in list(H.LIVE_SESSIONS):
            assert sess.verify_guards(), "a kernel wrote outside a device buffer of " + sess.wl.name
