import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs on the B200 box)")


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


@pytest.fixture(params=["pinned", "pageable", "mixed"])
def host_route(request, monkeypatch):
    """The host-buffer entry points accept page-locked and pageable host memory.  Tests that build their host
    buffers with Tensor.pin_memory() run three times: as written ("pinned"), with every buffer left pageable
    ("pageable"), and with the buffers pinned in runs of twelve ("mixed": calls with buffers of both kinds follow
    one another without a synchronisation)."""
    import torch
    if request.param == "pinned":
        return request.param
    real = torch.Tensor.pin_memory
    count = {"n": 0}

    def maybe_pin(self, *a, **kw):
        count["n"] += 1
        if request.param == "mixed" and (count["n"] // 12) % 2 == 0:
            return real(self, *a, **kw)
        return self.clone() if self.device.type == "cpu" else self.cpu()

    monkeypatch.setattr(torch.Tensor, "pin_memory", maybe_pin)
    return request.param
