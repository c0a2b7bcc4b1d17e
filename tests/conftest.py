import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on the GPU box)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, when no device is present (e.g. plain `pytest tests`)."""
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


class _GuardingTorch:
    """Stands in for the `torch` module inside the binding during GPU tests: every device buffer the
    binding allocates for the library to write (outputs, workspaces) gets a guard band on both sides,
    and the bands are checked when the test ends."""

    def __init__(self, real, registry):
        self._real = real
        self._registry = registry

    def __getattr__(self, name):
        return getattr(self._real, name)

    def _guarded(self, shape, dtype, device, fill=None):
        from parity_util import Guarded
        dtype = dtype or self._real.float32
        if device is None or self._real.device(device).type != "cuda":
            return None
        g = Guarded(tuple(shape), dtype, device, f"binding buffer {tuple(shape)} {dtype}")
        if fill is not None:
            g.view.fill_(fill)
        self._registry.append(g)
        return g.view

    def empty(self, *size, dtype=None, device=None, **kw):
        shape = size[0] if len(size) == 1 and isinstance(size[0], (tuple, list, self._real.Size)) else size
        t = self._guarded(shape, dtype, device)
        return t if t is not None else self._real.empty(*size, dtype=dtype, device=device, **kw)

    def zeros(self, *size, dtype=None, device=None, **kw):
        shape = size[0] if len(size) == 1 and isinstance(size[0], (tuple, list, self._real.Size)) else size
        t = self._guarded(shape, dtype, device, fill=0)
        return t if t is not None else self._real.zeros(*size, dtype=dtype, device=device, **kw)

    def empty_like(self, other, **kw):
        if kw or not other.is_contiguous():
            return self._real.empty_like(other, **kw)
        t = self._guarded(tuple(other.shape), other.dtype, other.device)
        return t if t is not None else self._real.empty_like(other)


@pytest.fixture(autouse=True)
def library_write_guards(request, monkeypatch):
    """GPU tests only: buffers the binding hands to the library sit between guard bands that must be
    untouched when the test ends (the stand-in for a memory checker on the library's writes)."""
    if "gpu" not in request.keywords:
        yield None
        return
    import torch
    if not torch.cuda.is_available():
        yield None
        return
    from paper_2609_34370_b200 import binding
    registry = []
    monkeypatch.setattr(binding, "torch", _GuardingTorch(torch, registry))
    yield registry
    torch.cuda.synchronize()
    for g in registry:
        g.check()
