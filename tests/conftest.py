import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


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
def guard_bands(request, monkeypatch):
    """Every GPU test runs with sentinel bands around the buffers the library writes: the output
    that Layer.forward allocates and the channel-split workspace.  After each forward the bands
    are checked, so a store one element past a plane fails the test that made it instead of
    landing silently in a neighbouring allocation."""
    if "gpu" not in request.keywords:
        yield
        return
    import torch
    from paper_1909_05073_b200 import binding as B
    from util import Guarded

    real_forward = B.Layer.forward

    def workspace(self, x_shape):
        n, _, h, w = x_shape
        need = B.pconv_workspace_bytes(self.handle, n, h, w)
        if need == 0:
            return None
        g = getattr(self, "_ws_guard", None)
        if g is None or g.nbytes < need:
            g = self._ws_guard = Guarded((need,), torch.uint8, fill=0)
            self._ws = g.t
        return g.t

    def forward(self, x, relu=True, kernel=0, out=None, split=False, pool=False):
        g = None
        if out is None:
            n, c, h, w = self.out_shape(x.shape)
            shape = (n, c, h // 2, w // 2) if pool else (n, c, h, w)
            g = Guarded(shape, x.dtype, fill=float("nan"))   # an element never written fails the comparison
            out = g.t
        y = real_forward(self, x, relu=relu, kernel=kernel, out=out, split=split, pool=pool)
        if g is not None:
            g.check("output of Layer.forward %s" % (tuple(x.shape),))
        wg = getattr(self, "_ws_guard", None)
        if wg is not None:
            wg.check("workspace of Layer.forward %s" % (tuple(x.shape),))
        return y

    monkeypatch.setattr(B.Layer, "workspace", workspace)
    monkeypatch.setattr(B.Layer, "forward", forward)
    yield
