import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


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


@pytest.fixture(autouse=True)
def _device_status_stays_clean(monkeypatch):
    """With HVD_ASSERT_DEVICE_STATUS=1 (set by the test that reruns the edge cases against the bounds-checked
    build of the library) every context must still report device status 0 when it is closed."""
    if os.environ.get("HVD_ASSERT_DEVICE_STATUS") != "1":
        yield
        return
    import paper_2606_01019_b200 as H
    orig = H.Context.close

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            assert self.hvd_device_status() == 0, "a kernel of the bounds-checked build recorded an index out of range"
        orig(self)

    monkeypatch.setattr(H.Context, "close", close)
    yield
