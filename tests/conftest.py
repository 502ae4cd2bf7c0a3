import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_report_header(config):
    try:
        from paper_2505_24544_b200 import binding
        return "beagle library: " + binding.load_library().beagle_version().decode()
    except Exception as e:          # not built yet: the tests that need it build it
        return f"beagle library: not loaded ({e})"


@pytest.fixture(autouse=True)
def device_status_after_gpu_test(request):
    """After every GPU test each open context must report a clean device status: no kernel abandoned a bounded wait and
    (bounds-checking build) no index check fired.  Tests that provoke the status on purpose consume it themselves."""
    yield
    if "gpu" not in request.keywords:
        return
    from paper_2505_24544_b200 import binding
    for ctx in list(binding.LIVE_CONTEXTS):
        if getattr(ctx, "handle", None):
            binding.beagle_check_device(ctx)


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
