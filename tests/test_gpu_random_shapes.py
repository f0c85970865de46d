"""GPU parity on seeded random layer shapes: the launch plan (warps per unit, channel splits, ring
depths, raw ring, tile widths) depends on the shape in many ways, so many small shapes are run
through the default path, with and without workspace and fused pool, against the CPU oracle."""
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


def random_case(rng):
    c_in = int(rng.choice([1, 3, 7, 8, 9, 16, 24, 40, 64, 100, 136]))
    c_out = int(rng.choice([1, 5, 16, 17, 32, 48, 80, 130]))
    h = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 13, 14, 16, 28, 33]))
    w = int(rng.choice([1, 2, 3, 4, 6, 7, 8, 14, 15, 16, 30, 32, 34, 65]))
    n = int(rng.choice([1, 1, 2, 3, 9]))
    stride = int(rng.choice([1, 1, 2]))
    keep = float(rng.choice([0.1, 0.3, 0.6, 1.0]))
    storage = str(rng.choice(["f32", "f32", "f16"]))
    patterns = synth.PATTERNS8 if rng.random() < 0.7 else synth.PATTERNS12
    return c_in, c_out, h, w, n, stride, keep, storage, patterns


@pytest.mark.parametrize("seed", range(48))
def test_random_shape_matches_the_oracle(seed):
    rng = np.random.default_rng(9000 + seed)
    c_in, c_out, h, w, n, stride, keep, storage, patterns = random_case(rng)
    spec = synth.LayerSpec("r", c_in, c_out, h, w, stride, keep, probs=(1 / len(patterns),) * len(patterns))
    wt, bias, _ = synth.gen_weights(spec, 9000 + seed, patterns)
    x = synth.gen_input(spec, n, 9000 + seed)
    layer = B.Layer(wt, patterns, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    ref = oracle.conv3x3(x, wt, bias, stride, True, storage)
    what = "seed %d: %s" % (seed, (c_in, c_out, h, w, n, stride, keep, storage, len(patterns)))
    for split in (False, True):
        y = layer.forward(xt, relu=True, split=split)
        torch.cuda.synchronize()
        check_close(y.float().cpu().numpy(), ref, storage, what + " split=%s" % split)
        if ref.shape[2] >= 2 and ref.shape[3] >= 2:
            yp = layer.forward(xt, relu=True, split=split, pool=True)
            torch.cuda.synchronize()
            check_close(yp.float().cpu().numpy(), oracle.maxpool2x2(ref), storage, what + " pooled split=%s" % split)
    ws = getattr(layer, "_ws", None)
    if ws is not None:
        assert not ws.any()
    assert B.pconv_device_status(layer.handle)[0] == 0
    layer.close()


@pytest.mark.parametrize("seed", range(32))
def test_random_shape_with_the_pinned_forms_matches_the_oracle(seed):
    """The same shapes through the forms a caller can pin: 8 rows per lane, the cluster reduction
    of the channel split and the bulk-copy staging, alone and together (canonical pattern sets;
    a form a shape cannot take must leave the result unchanged)."""
    rng = np.random.default_rng(9500 + seed)
    c_in, c_out, h, w, n, stride, keep, storage, _ = random_case(rng)
    if seed % 4 == 0:          # shapes whose rows or planes start on 16-byte boundaries
        h, w = int(rng.choice([4, 8, 14, 16, 28])), int(rng.choice([4, 8, 14, 16, 28, 36, 64]))
    spec = synth.LayerSpec("r", c_in, c_out, h, w, stride, keep)
    wt, bias, _ = synth.gen_weights(spec, 9500 + seed)
    x = synth.gen_input(spec, n, 9500 + seed)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    ref = oracle.conv3x3(x, wt, bias, stride, True, storage)
    pooled = oracle.maxpool2x2(ref) if ref.shape[2] >= 2 and ref.shape[3] >= 2 else None
    what = "seed %d: %s" % (seed, (c_in, c_out, h, w, n, stride, keep, storage))
    for flags in (B.ROWS8, B.CLUSTER, B.STAGE_BULK, B.ROWS8 | B.CLUSTER | B.STAGE_BULK):
        for split in (False, True):
            y = layer.forward(xt, relu=True, kernel=B.KERNEL_TILED | flags, split=split)
            check_close(y.float().cpu().numpy(), ref, storage, what + " flags %x split=%s" % (flags, split))
            if pooled is not None:
                yp = layer.forward(xt, relu=True, kernel=B.KERNEL_TILED | flags, split=split, pool=True)
                check_close(yp.float().cpu().numpy(), pooled, storage, what + " flags %x pooled split=%s" % (flags, split))
    ws = getattr(layer, "_ws", None)
    if ws is not None:
        assert not ws.any()
    assert B.pconv_device_status(layer.handle)[0] == 0
