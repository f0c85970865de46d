"""The entry point for callers that cannot allocate device memory (pconv_forward_static_ws).

Some users of this library run where cudaMalloc is off limits: inside another framework's memory
plan, under an allocator they do not own, or on a path that must never touch the driver's
allocator.  For them the channel-split scratch lives in a fixed array inside the library.  This
test calls that entry point through the C ABI twice in a row and checks each result against the
ordinary workspace entry point (pconv_forward_ws) and against the CPU oracle, with the tolerance
of the other parity tests.  It is collected last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import check_close

pytestmark = pytest.mark.gpu


def _layer(c_in, c_out, h, seed, stride=1):
    """(packed layer, device input, the CPU oracle's result for it)"""
    spec = synth.LayerSpec("t", c_in, c_out, h, h, stride, 0.35)
    w, b, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, 1, seed)
    return (B.Layer(w, synth.PATTERNS8, stride, B.F32, b), torch.from_numpy(x).cuda(),
            oracle.conv3x3(x, w, b, stride, True))


def test_static_workspace_entry_point_matches_the_workspace_entry_point():
    pbuild.build()
    layer, x, want = _layer(128, 96, 28, 31)
    assert 0 < B.pconv_workspace_bytes(layer.handle, 1, 28, 28) <= B.STATIC_WS_BYTES
    ref = layer.forward(x, relu=True, split=True)        # existing entry point, caller's buffer
    torch.cuda.synchronize()
    ref = ref.cpu().numpy()
    for call in range(2):                                 # two calls in a row share the array
        y = torch.full_like(torch.from_numpy(ref), float("nan")).cuda()
        B.pconv_forward_static_ws(layer.handle, x, layer.bias, y, B.RELU)
        torch.cuda.synchronize()
        check_close(y.cpu().numpy(), ref, "f32", "static workspace, call %d" % call)
        check_close(y.cpu().numpy(), want, "f32", "static workspace against the oracle, call %d" % call)
    # a different layer right after: leftovers of the previous shape must not matter
    layer2, x2, want2 = _layer(64, 64, 14, 32)
    ref2 = layer2.forward(x2, relu=True, split=True).cpu().numpy()
    y2 = torch.empty_like(torch.from_numpy(ref2)).cuda()
    B.pconv_forward_static_ws(layer2.handle, x2, layer2.bias, y2, B.RELU)
    torch.cuda.synchronize()
    check_close(y2.cpu().numpy(), ref2, "f32", "static workspace, second layer")
    check_close(y2.cpu().numpy(), want2, "f32", "static workspace against the oracle, second layer")
    assert B.pconv_device_status(layer.handle)[0] == 0
    layer.close()
    layer2.close()


def test_static_workspace_rejects_shapes_beyond_its_size():
    pbuild.build()
    # 128 filters on one 640x32 image: too few output tiles to fill the GPU, so a deep enough
    # layer has its channel range split across CTAs, and the partial sums (128*640*32*4 B =
    # 10.5 MB) do not fit the 8 MiB array.  The split is the library's choice: take the first depth
    # for which it is made.
    layer = None
    for c_in in (512, 1024, 2048):
        spec = synth.LayerSpec("t", c_in, 128, 640, 32, 1, 0.3)
        w, b, _ = synth.gen_weights(spec, 5)
        cand = B.Layer(w, synth.PATTERNS8, 1, B.F32, b)
        if B.pconv_workspace_bytes(cand.handle, 1, 640, 32) > B.STATIC_WS_BYTES:
            layer = cand
            break
        cand.close()
    assert layer is not None, "no tested depth makes the library split this shape"
    assert B.pconv_plan(layer.handle, 1, 640, 32, 0, True)["channel_splits"] > 1
    x = torch.zeros(1, c_in, 640, 32, device="cuda")
    y = torch.full((1, 128, 640, 32), 7.0, device="cuda")
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward_static_ws(layer.handle, x, layer.bias, y, B.RELU)
    assert e.value.status == 11 and "PCONV_ERR_WORKSPACE" in str(e.value)
    torch.cuda.synchronize()
    assert bool((y == 7.0).all())          # nothing was launched
    layer.close()
