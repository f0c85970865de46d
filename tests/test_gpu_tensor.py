"""GPU parity of the dense tensor-core path (fp16 storage, stride 1: zero-inserted weights as an
implicit GEMM on tcgen05.mma) against the CPU oracle, through the C ABI with the kernel pinned by
PCONV_KERNEL_TENSOR: shapes that cover every tile width (8, 16, 32 columns), several column tiles,
narrow maps that put several images side by side in a strip row, widths that are no multiple of 8
(element-wise loads), channel and filter counts that need zero padding, more tiles than SMs
(persistent CTAs, both accumulator buffers), and the library's own choice between this path and
the pattern-sparse kernel."""
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


CASES = [  # (c_in, c_out, h, w, n, keep)
    (16, 64, 32, 32, 2, 0.5),
    (64, 64, 32, 32, 4, 0.25),
    (3, 64, 32, 32, 3, 0.25),        # channels padded to 16; many filters without a kernel
    (40, 130, 16, 16, 5, 0.4),       # two filter tiles of 128, the second mostly padding
    (24, 48, 8, 8, 9, 0.5),
    (32, 32, 4, 4, 21, 0.5),         # two images side by side in a strip row
    (16, 16, 2, 2, 37, 0.6),         # four images side by side
    (4, 4, 1, 1, 70, 1.0),           # eight images side by side
    (8, 24, 3, 3, 10, 0.7),          # cells of width 4 holding 3 columns
    (8, 24, 14, 14, 3, 0.5),         # width not a multiple of 8: element-wise loads
    (8, 16, 7, 5, 4, 0.5),
    (5, 7, 3, 9, 2, 0.8),
    (16, 32, 6, 40, 2, 0.4),         # two column tiles of 32, the second ragged
    (16, 32, 5, 72, 1, 0.4),         # three column tiles
    (32, 256, 8, 8, 6, 0.3),         # two full filter tiles
    (48, 64, 32, 32, 40, 0.25),      # 330 pixel tiles: more than one per CTA
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_tensor_path_matches_the_oracle(case):
    c_in, c_out, h, w, n, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, 1, keep)
    seed = 4000 + c_in * 13 + c_out + h * 3 + w
    wt, bias, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F16, bias)
    xt = torch.from_numpy(x).cuda().half()
    for relu in (True, False):
        got = layer.forward(xt, relu=relu, kernel=B.KERNEL_TENSOR)
        ref = oracle.conv3x3(x, wt, bias, 1, relu, "f16")
        check_close(got.float().cpu().numpy(), ref, "f16", "%s relu=%s" % (case, relu))
    # the same result as the pattern-sparse kernel up to summation order and the fp16 store
    tiled = layer.forward(xt, relu=True, kernel=B.KERNEL_TILED).float().cpu().numpy()
    dense = layer.forward(xt, relu=True, kernel=B.KERNEL_TENSOR).float().cpu().numpy()
    assert np.abs(tiled - dense).max() <= 2e-3 * (1 + np.abs(tiled).max())
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


@pytest.mark.parametrize("case", [(512, 256, 2, 2, 64, 0.25), (256, 130, 4, 4, 40, 0.3), (192, 64, 8, 8, 12, 0.4)],
                         ids=lambda c: "x".join(str(v) for v in c))
def test_tensor_path_with_the_channel_steps_split_across_ctas(case):
    """Few pixel tiles, deep layer: with a workspace the channel steps of a tile are cut in parts
    that different CTAs take; the parts meet in fp32 sums in the workspace, which must be zero
    again afterwards (two forwards in a row use it)."""
    c_in, c_out, h, w, n, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, 1, keep)
    wt, bias, _ = synth.gen_weights(spec, 555 + c_in)
    x = synth.gen_input(spec, n, 555 + c_in)
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F16, bias)
    assert B.pconv_workspace_bytes(layer.handle, n, h, w) > 0
    xt = torch.from_numpy(x).cuda().half()
    ref = oracle.conv3x3(x, wt, bias, 1, True, "f16")
    for rep in range(2):
        got = layer.forward(xt, relu=True, kernel=B.KERNEL_TENSOR, split=True)
        check_close(got.float().cpu().numpy(), ref, "f16", "%s split, call %d" % (case, rep))
        assert not layer._ws.any()
    same = layer.forward(xt, relu=True, kernel=B.KERNEL_TENSOR, split=False)       # no workspace: no split
    check_close(same.float().cpu().numpy(), ref, "f16", "%s unsplit" % (case,))
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


def test_tensor_path_without_bias_and_with_twelve_patterns():
    spec = synth.LayerSpec("t", 32, 48, 16, 16, 1, 0.4, probs=(1 / 12,) * 12)
    wt, _, _ = synth.gen_weights(spec, 91, synth.PATTERNS12)
    x = synth.gen_input(spec, 3, 91)
    layer = B.Layer(wt, synth.PATTERNS12, 1, B.F16, None)
    got = layer.forward(torch.from_numpy(x).cuda().half(), relu=False, kernel=B.KERNEL_TENSOR)
    check_close(got.float().cpu().numpy(), oracle.conv3x3(x, wt, None, 1, False, "f16"), "f16", "12 patterns")
    layer.close()


def test_tensor_path_is_refused_where_it_does_not_apply():
    spec = synth.LayerSpec("t", 16, 16, 8, 8, 1, 0.5)
    wt, bias, _ = synth.gen_weights(spec, 3)
    x = torch.from_numpy(synth.gen_input(spec, 2, 3)).cuda()
    f32 = B.Layer(wt, synth.PATTERNS8, 1, B.F32, bias)
    with pytest.raises(B.PconvError) as e:
        f32.forward(x, kernel=B.KERNEL_TENSOR)
    assert "PCONV_ERR_UNSUPPORTED" in str(e.value)
    s2 = B.Layer(wt, synth.PATTERNS8, 2, B.F16, bias)
    with pytest.raises(B.PconvError):
        s2.forward(x.half(), kernel=B.KERNEL_TENSOR)
    f16 = B.Layer(wt, synth.PATTERNS8, 1, B.F16, bias)
    with pytest.raises(B.PconvError):
        f16.forward(x.half(), kernel=B.KERNEL_TENSOR, pool=True)     # no fused pool on this path
    for l in (f32, s2, f16):
        l.close()


def test_the_library_picks_the_tensor_path_for_large_fp16_batches_only():
    spec = synth.LayerSpec("t", 64, 64, 32, 32, 1, 0.25)
    wt, bias, _ = synth.gen_weights(spec, 8)
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F16, bias)
    assert B.pconv_plan(layer.handle, 256, 32, 32)["tensor_path"] == 1
    assert B.pconv_plan(layer.handle, 1, 32, 32)["tensor_path"] == 0       # too few tiles for the device
    f32 = B.Layer(wt, synth.PATTERNS8, 1, B.F32, bias)
    assert B.pconv_plan(f32.handle, 256, 32, 32)["tensor_path"] == 0
    # default forward of a large batch = the pinned tensor kernel, bit for bit (it is deterministic)
    x = torch.from_numpy(synth.gen_input(spec, 64, 8)).cuda().half()
    a = layer.forward(x, relu=True)
    b = layer.forward(x, relu=True, kernel=B.KERNEL_TENSOR)
    assert torch.equal(a, b)
    layer.close()
    f32.close()


def test_stack_with_tensor_layers_and_separate_pools_matches_the_oracle():
    specs = [synth.LayerSpec("a", 16, 64, 16, 16, 1, 0.4, pool_after=True),
             synth.LayerSpec("b", 64, 64, 8, 8, 1, 0.4),
             synth.LayerSpec("c", 64, 32, 8, 8, 1, 0.4, pool_after=True)]
    n = 160
    ws, layers = [], []
    for i, s in enumerate(specs):
        w, b, _ = synth.gen_weights(s, 70 + i)
        ws.append((w, b))
        layers.append(B.Layer(w, synth.PATTERNS8, 1, B.F16, b))
    assert all(B.pconv_plan(l.handle, n, s.h, s.w)["tensor_path"] == 1 for l, s in zip(layers, specs))
    x = synth.gen_input(specs[0], n, 70)
    a = x
    for (w, b), s in zip(ws, specs):
        a = oracle.conv3x3(a, w, b, 1, True, "f16").astype(np.float16).astype(np.float32)
        if s.pool_after:
            a = oracle.maxpool2x2(a)
    stack = B.Stack(layers, [s.pool_after for s in specs], n, 16, 16, B.RELU)
    y = torch.empty(stack.out_shape, dtype=torch.float16, device="cuda")
    stack.forward(torch.from_numpy(x).cuda().half(), y)
    torch.cuda.synchronize()
    check_close(y.float().cpu().numpy(), a, "f16", "stack of tensor-path layers")
    assert stack.status() == (0, 0)
    stack.close()
