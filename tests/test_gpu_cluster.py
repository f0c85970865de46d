"""GPU parity of the cluster form of the channel split (PCONV_CLUSTER: the thread blocks that share
an output tile add their partial sums up through distributed shared memory) against the CPU
oracle: cluster sizes 2 to 16, both row forms of the kernel, fp16 storage, stride 2 and the fused
max-pool; the workspace must stay untouched, and a shape the cluster form cannot take must fall
back to the workspace form with the same result."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import check_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()
    B.lib()


CASES = [  # (c_in, c_out, h, w, n, stride, keep, storage, pool, extra flags)
    (256, 256, 56, 56, 1, 1, 0.3, "f32", False, 0),        # 2 CTAs per tile
    (512, 512, 28, 28, 1, 1, 0.3, "f32", True, 0),         # 4 CTAs per tile, pooled
    (512, 512, 14, 14, 1, 1, 0.3, "f32", False, 0),        # 16 CTAs per tile (beyond the portable size)
    (256, 130, 14, 14, 2, 1, 0.4, "f16", False, 0),        # padding filters in the last group
    (128, 96, 28, 28, 1, 2, 0.5, "f32", False, 0),
    (128, 128, 20, 24, 1, 1, 0.3, "f32", False, B.ROWS8),
    (64, 64, 56, 56, 1, 1, 0.3, "f16", True, B.ROWS8),
    (40, 24, 9, 5, 3, 2, 0.5, "f16", False, 0),
    (2048, 32, 7, 7, 1, 1, 0.2, "f32", False, 0),          # more splits than a cluster holds: falls back
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_cluster_split_matches_the_oracle(case):
    c_in, c_out, h, w, n, stride, keep, storage, pool, extra = case
    spec = synth.LayerSpec("cl", c_in, c_out, h, w, stride, keep)
    seed = 9100 + c_in + 3 * c_out + h
    wt, bias, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    plan = B.pconv_plan(layer.handle, n, h, w, extra, True)
    ref = oracle.conv3x3(x, wt, bias, stride, True, storage)
    if pool:
        ref = oracle.maxpool2x2(ref)
    ws = layer.workspace(xt.shape)
    got = None
    for _ in range(3):
        got = layer.forward(xt, relu=True, kernel=B.KERNEL_TILED | B.CLUSTER | extra, split=True, pool=pool)
        check_close(got.float().cpu().numpy(), ref, storage, "%s plan %s" % (case, plan))
    if ws is not None:
        assert not ws.any()       # untouched by the cluster form, left zeroed by the workspace form
    other = layer.forward(xt, relu=True, kernel=B.KERNEL_TILED | extra, split=True, pool=pool)
    tol = 2e-2 if storage == "f16" else 1e-5
    assert np.abs(got.float().cpu().numpy() - other.float().cpu().numpy()).max() <= tol * (1 + np.abs(ref).max())
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


def test_cluster_stack_matches_the_plain_stack():
    cfg = synth.config(2)
    layers = []
    for li, spec in enumerate(cfg.layers[7:13]):     # the 28x28 and 14x14 layers of the VGG stack
        wt, b, _ = synth.gen_weights(spec, synth.layer_seed(2, 7 + li), cfg.patterns)
        layers.append(B.Layer(wt, cfg.patterns, spec.stride, B.F32, b))
    pools = [s.pool_after for s in cfg.layers[7:13]]
    s0 = cfg.layers[7]
    x = torch.from_numpy(synth.gen_input(s0, 1, 3)).cuda()
    outs = []
    for flags in (B.RELU, B.RELU | B.CLUSTER):
        stack = B.Stack(layers, pools, 1, s0.h, s0.w, flags)
        y = torch.empty(stack.out_shape, dtype=torch.float32, device="cuda")
        for _ in range(2):
            stack.forward(x, y)
        torch.cuda.synchronize()
        assert stack.status() == (0, 0)
        outs.append(y.cpu().numpy())
    assert np.abs(outs[0] - outs[1]).max() <= 1e-5 * (1 + np.abs(outs[0]).max())
