"""GPU parity of the tiled kernel's 8-rows-per-lane form (eight consumer warps, 256 Tensor-Memory
columns each, 32 packed FMAs per decoded kernel) against the CPU oracle, through the C ABI with
the form pinned by PCONV_ROWS8: both strides and storages, every tile width, the fused max-pool,
the channel split through the workspace (both warps-per-unit plans), ragged rows and columns, and
the planner's own choice between the two forms."""
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


CASES = [  # (c_in, c_out, h, w, n, stride, keep, storage, split, pool)
    (24, 40, 37, 45, 2, 1, 0.4, "f32", False, False),
    (24, 40, 37, 45, 2, 2, 0.4, "f32", False, False),
    (24, 40, 37, 45, 2, 1, 0.4, "f16", False, False),    # odd width: element-wise fp16 staging
    (24, 40, 36, 44, 2, 1, 0.4, "f16", False, True),     # even width: the raw ring; pooled
    (24, 40, 37, 45, 2, 1, 0.4, "f32", True, True),
    (64, 64, 56, 56, 1, 1, 0.3, "f32", True, False),     # batch 1: channel split, two warps per unit
    (128, 128, 14, 14, 3, 1, 0.3, "f32", True, False),   # 16-wide sub-tiles, 14 rows in two blocks of 8
    (128, 128, 7, 7, 5, 1, 0.3, "f32", True, False),
    (64, 96, 28, 28, 2, 2, 0.5, "f32", True, False),
    (64, 96, 29, 27, 2, 2, 0.5, "f16", False, False),
    (3, 64, 64, 64, 1, 1, 1.0, "f32", False, True),
    (16, 16, 4, 4, 9, 1, 0.5, "f32", False, False),
    (16, 16, 2, 2, 33, 1, 0.5, "f16", False, False),
    (40, 24, 9, 5, 3, 2, 0.5, "f16", True, False),
    (16, 48, 8, 300, 1, 1, 0.5, "f32", False, False),    # ten column tiles, one block of rows
    (8, 16, 65, 9, 2, 1, 0.7, "f32", False, True),       # nine row blocks, the last with one row
    (256, 64, 16, 16, 40, 1, 0.5, "f32", False, False),  # more tiles than SMs
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_eight_rows_per_lane_matches_the_oracle(case):
    c_in, c_out, h, w, n, stride, keep, storage, split, pool = case
    spec = synth.LayerSpec("r8", c_in, c_out, h, w, stride, keep)
    seed = 8000 + c_in * 7 + c_out + h * 5 + w
    wt, bias, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    plan = B.pconv_plan(layer.handle, n, h, w, B.ROWS8, split)
    assert plan["rows_per_lane"] == 8 and plan["warps_per_unit"] in (1, 2)
    assert plan["groups_per_cta"] * plan["pixel_sets"] * plan["warps_per_unit"] <= 8
    for relu in (True, False):
        ref = oracle.conv3x3(x, wt, bias, stride, relu, storage)
        if pool:
            ref = oracle.maxpool2x2(ref)
        for _ in range(2):     # twice: a split launch must leave its workspace and tickets zeroed
            got = layer.forward(xt, relu=relu, kernel=B.KERNEL_TILED | B.ROWS8, split=split, pool=pool)
            check_close(got.float().cpu().numpy(), ref, storage, "%s relu=%s" % (case, relu))
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


def test_eight_rows_reproducible_mode_is_bit_identical():
    spec = synth.LayerSpec("r8", 96, 48, 20, 24, 1, 0.4)
    wt, bias, _ = synth.gen_weights(spec, 77)
    x = torch.from_numpy(synth.gen_input(spec, 1, 77)).cuda()
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F32, bias)
    outs = [layer.forward(x, kernel=B.KERNEL_TILED | B.ROWS8 | B.REPRODUCIBLE).cpu().numpy() for _ in range(4)]
    for o in outs[1:]:
        assert np.array_equal(o, outs[0])
    check_close(outs[0], oracle.conv3x3(x.cpu().numpy(), wt, bias, 1, True), "f32", "reproducible")
    layer.close()


def test_planner_takes_eight_rows_for_large_batches_only():
    """Measured: the 8-row form wins where a warp owns its unit's whole channel range (large
    batches) and loses where channels are split among warps or CTAs (batch 1)."""
    big = synth.config(5)
    spec = big.layers[0]
    wt, bias, _ = synth.gen_weights(spec, synth.layer_seed(5, 0), big.patterns)
    layer = B.Layer(wt, big.patterns, spec.stride, B.F32, bias)
    p = B.pconv_plan(layer.handle, big.batch, spec.h, spec.w, 0, True)
    assert p["rows_per_lane"] == 8 and p["warps_per_unit"] == 1 and p["channel_splits"] == 1
    p1 = B.pconv_plan(layer.handle, 1, spec.h, spec.w, 0, True)
    assert p1["rows_per_lane"] == 4
    assert B.pconv_plan(layer.handle, 1, spec.h, spec.w, B.ROWS4, True)["rows_per_lane"] == 4
    layer.close()


def test_eight_rows_refused_where_it_does_not_exist():
    spec = synth.LayerSpec("r8", 16, 16, 12, 12, 1, 0.5)
    x = torch.from_numpy(synth.gen_input(spec, 1, 5)).cuda()
    wt, bias, _ = synth.gen_weights(spec, 5, synth.PATTERNS12)
    layer = B.Layer(wt, synth.PATTERNS12, 1, B.F32, bias)     # two-byte codes: 4 rows per lane only
    with pytest.raises(B.PconvError):
        layer.forward(x, kernel=B.KERNEL_TILED | B.ROWS8)
    y = layer.forward(x, kernel=B.KERNEL_TILED | B.ROWS4)
    check_close(y.cpu().numpy(), oracle.conv3x3(x.cpu().numpy(), wt, bias, 1, True), "f32", "rows4 wide")
    layer.close()
    wt, bias, _ = synth.gen_weights(spec, 5)
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F32, bias)
    for bad in (B.KERNEL_GENERIC_TAPS | B.ROWS8, B.ROWS4 | B.ROWS8):
        with pytest.raises(B.PconvError):
            layer.forward(x, kernel=bad)
    layer.close()
