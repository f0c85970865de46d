"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same
seeded inputs -- element by element, at sizes that span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import check_close

pytestmark = pytest.mark.gpu

KERNELS = {"simple": B.KERNEL_SIMPLE, "tiled": B.KERNEL_TILED, "generic": B.KERNEL_GENERIC_TAPS,
           "auto": 0}


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()
    B.lib()


def run_layer(w, bias, x, stride=1, storage="f32", relu=True, kernel="auto", patterns=None):
    st = B.F16 if storage == "f16" else B.F32
    layer = B.Layer(w, patterns or synth.PATTERNS8, stride, st, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    y = layer.forward(xt, relu=relu, kernel=KERNELS[kernel])
    torch.cuda.synchronize()
    status, where = B.pconv_device_status(layer.handle)
    assert status == 0, ("device status", status, where)
    layer.close()
    return y.float().cpu().numpy()


def oracle_layer(w, bias, x, stride=1, storage="f32", relu=True):
    return oracle.conv3x3(x, w, bias, stride, relu, storage)


SMALL = [  # (c_in, c_out, h, w, n, stride, keep)
    (1, 1, 1, 1, 1, 1, 1.0),
    (3, 5, 5, 7, 2, 1, 0.7),
    (5, 17, 9, 9, 3, 1, 0.5),
    (9, 33, 6, 35, 2, 1, 0.4),      # one column past a 32-wide tile
    (16, 16, 37, 33, 1, 1, 0.3),
    (20, 40, 14, 14, 2, 1, 0.35),
    (8, 24, 7, 7, 5, 1, 0.5),
    (4, 16, 2, 2, 9, 1, 0.6),
    (7, 19, 4, 4, 6, 1, 0.5),
    (3, 5, 5, 7, 2, 2, 0.7),
    (12, 20, 28, 28, 2, 2, 0.4),
    (16, 32, 14, 14, 3, 2, 0.35),
    (6, 16, 9, 11, 2, 2, 0.5),
    (5, 8, 1, 9, 2, 2, 0.8),
]


@pytest.mark.parametrize("kernel", ["simple", "tiled", "generic", "auto"])
@pytest.mark.parametrize("storage", ["f32", "f16"])
@pytest.mark.parametrize("case", SMALL, ids=lambda c: "x".join(str(v) for v in c))
def test_small_layers_match_the_oracle(case, storage, kernel):
    c_in, c_out, h, w, n, stride, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, stride, keep)
    seed = 1000 + c_in * 7 + c_out + h
    wt, bias, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    for relu in (True, False):
        got = run_layer(wt, bias, x, stride, storage, relu, kernel)
        ref = oracle_layer(wt, bias, x, stride, storage, relu)
        check_close(got, ref, storage, "%s relu=%s" % (case, relu))


@pytest.mark.parametrize("kernel", ["simple", "tiled", "generic"])
def test_config1_full_layer(kernel):
    cfg = synth.config(1)
    spec = cfg.layers[0]
    wt, bias, _ = synth.gen_weights(spec, synth.layer_seed(1, 0))
    x = synth.gen_input(spec, cfg.batch, synth.layer_seed(1, 0))
    got = run_layer(wt, bias, x, kernel=kernel)
    check_close(got, oracle_layer(wt, bias, x), "f32", "config 1")


@pytest.mark.parametrize("kernel", ["simple", "tiled", "generic"])
@pytest.mark.parametrize("stride", [1, 2])
def test_single_tap_shift_through_the_gpu(kernel, stride):
    """Each of the 9 taps alone is a sub-support of some pattern (non-strict packing), and the
    output must be the shifted, zero-filled input exactly."""
    rng = np.random.default_rng(4)
    h, w = 9, 13
    x = rng.normal(size=(1, 3, h, w)).astype(np.float32)
    for t in range(9):
        wt = np.zeros((2, 3, 3, 3), np.float32)
        wt[1, 2, t // 3, t % 3] = 1.0
        got = run_layer(wt, None, x, stride, "f32", False, kernel)
        ref = oracle_layer(wt, None, x, stride, "f32", False)
        assert np.array_equal(got, ref), t
        assert not got[:, 0].any()


@pytest.mark.parametrize("kernel", ["simple", "tiled", "generic"])
def test_empty_filters_and_no_bias(kernel):
    spec = synth.LayerSpec("t", 6, 20, 10, 10, 1, 0.5)
    wt, bias, _ = synth.gen_weights(spec, 77)
    wt[3] = 0
    wt[17] = 0
    x = synth.gen_input(spec, 2, 77)
    got = run_layer(wt, bias, x, kernel=kernel)
    check_close(got, oracle_layer(wt, bias, x), "f32", "empty filters")
    assert np.allclose(got[:, 3], max(bias[3], 0.0))
    allzero = np.zeros_like(wt)
    got = run_layer(allzero, None, x, relu=False, kernel=kernel)
    assert not got.any()


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("kernel", ["simple", "tiled", "generic", "auto"])
def test_twelve_patterns_and_noncanonical_sets(kernel, stride):
    spec = synth.LayerSpec("t", 24, 40, 18, 21, stride, 0.4, probs=(1 / 12,) * 12)
    wt, bias, ids = synth.gen_weights(spec, 5, synth.PATTERNS12)
    assert ids.max() == 11
    x = synth.gen_input(spec, 2, 5)
    got = run_layer(wt, bias, x, stride=stride, kernel=kernel, patterns=synth.PATTERNS12)
    check_close(got, oracle_layer(wt, bias, x, stride), "f32", "12 patterns")


def all_masks_with_four_taps():
    return [m for m in range(512) if bin(m).count("1") == 4]


@pytest.mark.parametrize("stride", [1, 2])
def test_every_one_of_the_126_masks_has_a_correct_body(stride):
    """The tiled kernel holds one straight-line body per 4-of-9 mask: run them all, 14 masks to a
    layer (pattern sets hold at most 16), every kernel carrying one tap weight per tap."""
    masks = all_masks_with_four_taps()
    assert len(masks) == 126
    rng = np.random.default_rng(126 + stride)
    for lo in range(0, len(masks), 14):
        pats = tuple(masks[lo:lo + 14])
        c_in, c_out, h, w, n = 10, 2 * len(pats), 9, 13, 2
        wt = np.zeros((c_out, c_in, 3, 3), np.float32)
        for o in range(c_out):
            for c in range(c_in):
                if rng.random() < 0.6:
                    m = pats[(o + c) % len(pats)]
                    for t in range(9):
                        if m >> t & 1:
                            wt[o, c, t // 3, t % 3] = rng.uniform(0.5, 1.5) * rng.choice([-1.0, 1.0])
        bias = rng.normal(0, 0.1, c_out).astype(np.float32)
        x = rng.uniform(-1, 1, (n, c_in, h, w)).astype(np.float32)
        got = run_layer(wt, bias, x, stride=stride, kernel="tiled", patterns=pats)
        check_close(got, oracle_layer(wt, bias, x, stride), "f32", "masks %d.." % lo)


@pytest.mark.parametrize("storage", ["f32", "f16"])
def test_pack_unpack_round_trip_and_stats(storage):
    for cid in (1, 3, 5):
        cfg = synth.config(cid)
        spec = cfg.layers[-1]
        wt, bias, ids = synth.gen_weights(spec, synth.layer_seed(cid, 0))
        layer = B.Layer(wt, cfg.patterns, spec.stride, B.F16 if storage == "f16" else B.F32,
                        strict4=True)
        back = layer.unpack()
        expect = wt if storage == "f32" else wt.astype(np.float16).astype(np.float32)
        assert np.array_equal(back, expect)
        s = layer.stats()
        kept = ids >= 0
        assert s.kept_kernels == kept.sum()
        assert sum(s.per_pattern[:8]) == s.kept_kernels
        assert [s.per_pattern[p] for p in range(8)] == [(ids == p).sum() for p in range(8)]
        assert s.min_per_filter == kept.sum(1).min() and s.max_per_filter == kept.sum(1).max()
        assert s.canonical_patterns == 1
        perm = B.pconv_filter_order(layer.handle)
        assert sorted(perm[perm >= 0]) == list(range(spec.c_out))
        # reorder balances groups: heaviest group within a few kernels of the lightest
        assert s.max_group_kernels - s.min_group_kernels <= max(16, 0.05 * s.max_group_kernels)
        layer.close()


def test_fp16_rounding_matches_ieee():
    vals = np.concatenate([
        np.random.default_rng(0).normal(0, 1, 2000), np.random.default_rng(1).normal(0, 1e-5, 2000),
        np.array([65504.0, 65519.9, 6.1e-5, 5.96e-8, 2.98e-8, 2.9e-8, 3.1e-8, 1e-9, -0.0,
                  1.0009765625, 1.00048828125, 1.00146484375])]).astype(np.float32)
    n = (len(vals) + 3) // 4
    wt = np.zeros((1, n, 3, 3), np.float32)
    pos = [(0, 1), (1, 0), (1, 1), (1, 2)]       # pattern id 0
    flat = np.resize(vals, 4 * n)
    for c in range(n):
        for s, (u, v) in enumerate(pos):
            wt[0, c, u, v] = flat[4 * c + s]
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F16)
    assert np.array_equal(layer.unpack(), wt.astype(np.float16).astype(np.float32))
    layer.close()


def test_forward_argument_errors():
    spec = synth.LayerSpec("t", 4, 4, 8, 8, 1, 0.5)
    wt, bias, _ = synth.gen_weights(spec, 1)
    layer = B.Layer(wt, synth.PATTERNS8)
    x = torch.zeros(1, 4, 8, 8, device="cuda")
    y = torch.zeros(1, 4, 8, 8, device="cuda")
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward(layer.handle, x, None, y, flags=0x40000)   # an unknown bit
    assert e.value.status == 6
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward(layer.handle, x, None, y, flags=B.KERNEL_SIMPLE | B.KERNEL_TILED)
    assert e.value.status == 6
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward(layer.handle, x, None, x)                    # aliasing
    assert e.value.status == 2
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward(layer.handle, x.view(-1)[1:].view(-1)[:252].view(1, 4, 7, 9), None, y)
    assert e.value.status == 7                                       # misaligned x
    layer.close()


@pytest.mark.parametrize("storage", ["f32", "f16"])
def test_maxpool_matches_the_oracle(storage):
    rng = np.random.default_rng(9)
    for shape in [(2, 3, 8, 6), (1, 5, 7, 9), (3, 2, 2, 2)]:
        x = rng.normal(size=shape).astype(np.float32)
        xt = torch.from_numpy(x).cuda()
        if storage == "f16":
            xt = xt.half()
            x = xt.float().cpu().numpy()
        y = torch.empty(shape[0], shape[1], shape[2] // 2, shape[3] // 2, dtype=xt.dtype,
                        device="cuda")
        B.pconv_maxpool2x2(xt, y)
        assert np.array_equal(y.float().cpu().numpy(), oracle.maxpool2x2(x))


SPLIT_CASES = [  # batch-1 layers that the library splits over input channels when given a workspace
    (64, 64, 14, 14, 1, 1, 0.4), (128, 96, 28, 28, 1, 1, 0.3), (96, 160, 7, 7, 2, 1, 0.35),
    (72, 48, 28, 28, 1, 2, 0.4), (256, 64, 9, 11, 1, 1, 0.3),
]


@pytest.mark.parametrize("storage", ["f32", "f16"])
@pytest.mark.parametrize("case", SPLIT_CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_channel_split_path_matches_the_oracle(case, storage):
    c_in, c_out, h, w, n, stride, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, stride, keep)
    wt, bias, _ = synth.gen_weights(spec, 4242 + c_in)
    x = synth.gen_input(spec, n, 4242 + c_in)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    assert B.pconv_workspace_bytes(layer.handle, n, h, w) > 0
    ref = oracle_layer(wt, bias, x, stride, storage, True)
    for _ in range(3):   # the workspace must come back zeroed: repeated calls stay correct
        y = layer.forward(xt, relu=True, split=True)
        torch.cuda.synchronize()
        check_close(y.float().cpu().numpy(), ref, storage, "split %s" % (case,))
    assert not layer._ws.any()
    assert B.pconv_device_status(layer.handle)[0] == 0
    layer.close()


POOL_CASES = [  # (c_in, c_out, h, w, n, stride, keep): even and odd maps, narrow tiles, stride 2
    (8, 24, 12, 12, 2, 1, 0.5), (6, 20, 9, 11, 2, 1, 0.6), (16, 16, 37, 33, 1, 1, 0.3),
    (12, 40, 4, 4, 5, 1, 0.5), (12, 20, 28, 28, 2, 2, 0.4), (128, 96, 28, 28, 1, 1, 0.3),
    (256, 64, 14, 14, 1, 1, 0.3), (5, 8, 2, 3, 3, 1, 0.8),
]


@pytest.mark.parametrize("storage", ["f32", "f16"])
@pytest.mark.parametrize("kernel", ["tiled", "generic", "auto"])
@pytest.mark.parametrize("case", POOL_CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_fused_maxpool_matches_conv_then_pool(case, kernel, storage):
    c_in, c_out, h, w, n, stride, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, stride, keep)
    wt, bias, _ = synth.gen_weights(spec, 31 + c_in)
    x = synth.gen_input(spec, n, 31 + c_in)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F16 if storage == "f16" else B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    for relu in (True, False):
        ref = oracle.maxpool2x2(oracle_layer(wt, bias, x, stride, storage, relu))
        for split in (False, True):
            y = layer.forward(xt, relu=relu, kernel=KERNELS[kernel], split=split, pool=True)
            torch.cuda.synchronize()
            assert tuple(y.shape) == ref.shape
            check_close(y.float().cpu().numpy(), ref, storage, "fused pool %s relu=%s split=%s" % (case, relu, split))
    ws = getattr(layer, "_ws", None)
    if ws is not None:
        assert not ws.any()
    assert B.pconv_device_status(layer.handle)[0] == 0
    layer.close()


def test_fused_maxpool_is_refused_where_it_cannot_run():
    spec = synth.LayerSpec("t", 4, 8, 6, 6, 1, 0.5)
    wt, bias, _ = synth.gen_weights(spec, 5)
    layer = B.Layer(wt, synth.PATTERNS8, 1, B.F32, bias)
    x = torch.zeros(1, 4, 6, 6, device="cuda")
    with pytest.raises(B.PconvError) as e:
        layer.forward(x, kernel=B.KERNEL_SIMPLE, pool=True)
    assert "PCONV_ERR_UNSUPPORTED" in str(e.value)
    x1 = torch.zeros(1, 4, 1, 6, device="cuda")          # a one-row map cannot be pooled
    with pytest.raises(B.PconvError) as e:
        B.pconv_forward(layer.handle, x1, layer.bias, torch.zeros(1, 8, 1, 3, device="cuda"), B.POOL2X2)
    assert "PCONV_ERR_SHAPE" in str(e.value)
    layer.close()


@pytest.mark.parametrize("case", [(64, 128, 56, 56, 1, 1, 0.3), (256, 256, 14, 14, 1, 1, 0.3),
                                  (128, 128, 28, 28, 2, 2, 0.35), (512, 512, 7, 7, 1, 1, 0.3)],
                         ids=lambda c: "x".join(str(v) for v in c))
def test_reproducible_flag_gives_bit_identical_runs(case):
    c_in, c_out, h, w, n, stride, keep = case
    spec = synth.LayerSpec("t", c_in, c_out, h, w, stride, keep)
    wt, bias, _ = synth.gen_weights(spec, 55 + c_in)
    x = synth.gen_input(spec, n, 55 + c_in)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F32, bias)
    assert B.pconv_plan(layer.handle, n, h, w, 0, False)["warps_per_unit"] > 1   # several warps share a tile
    xt = torch.from_numpy(x).cuda()
    ws = layer.workspace(xt.shape)
    ref = oracle_layer(wt, bias, x, stride, "f32", True)
    first = None
    for _ in range(6):
        y = torch.empty(layer.out_shape(xt.shape), device="cuda")
        B.pconv_forward(layer.handle, xt, layer.bias, y, B.RELU | B.REPRODUCIBLE, workspace=ws)
        torch.cuda.synchronize()
        got = y.cpu().numpy()
        check_close(got, ref, "f32", "reproducible %s" % (case,))
        if first is None:
            first = got
        assert np.array_equal(got, first)
    if ws is not None:
        assert not ws.any()            # the flag keeps the channel range in one thread block
    assert B.pconv_device_status(layer.handle)[0] == 0
    layer.close()


PLAN_CASES = [  # shapes that make the library use each way of sharing the consumer warps
    (16, 128, 32, 32, 74, 1, 0.5),    # as many tiles as SMs: one warp per unit
    (64, 64, 224, 224, 1, 1, 0.3),    # one large image
    (64, 128, 112, 112, 1, 1, 0.3),
    (256, 256, 14, 14, 1, 1, 0.3),    # deep and small: warps share units and CTAs share tiles
    (128, 128, 56, 56, 1, 2, 0.3),
]


def test_every_warp_sharing_plan_matches_the_oracle():
    seen = set()
    for case in PLAN_CASES:
        c_in, c_out, h, w, n, stride, keep = case
        spec = synth.LayerSpec("t", c_in, c_out, h, w, stride, keep)
        wt, bias, _ = synth.gen_weights(spec, 777 + c_in)
        x = synth.gen_input(spec, n, 777 + c_in)
        layer = B.Layer(wt, synth.PATTERNS8, stride, B.F32, bias)
        xt = torch.from_numpy(x).cuda()
        ref = oracle_layer(wt, bias, x, stride, "f32", True)
        for with_ws in (False, True):
            plan = B.pconv_plan(layer.handle, n, h, w, 0, with_ws)
            assert plan["generic_taps"] == 0 and plan["warps_per_unit"] in (1, 2, 4)
            assert plan["smem_bytes"] <= 227 * 1024 and plan["stages"] >= 1
            # (the workspace size covers the pinned forms too, so it may be non-zero where the
            # planner's own choice does not split)
            assert plan["channel_splits"] == 1 or (with_ws and B.pconv_workspace_bytes(layer.handle, n, h, w) > 0)
            seen.add((plan["warps_per_unit"], plan["channel_splits"] > 1))
            for _ in range(2):
                y = layer.forward(xt, relu=True, split=with_ws)
                torch.cuda.synchronize()
                check_close(y.float().cpu().numpy(), ref, "f32", "plan %s of %s" % (plan, case))
        assert B.pconv_device_status(layer.handle)[0] == 0
        layer.close()
    assert {z for z, _ in seen} == {1, 2, 4}, seen
    assert (4, True) in seen and (4, False) in seen, seen


@pytest.mark.parametrize("storage", ["f32", "f16"])
def test_stack_matches_the_chained_oracle(storage):
    chans = [(3, 16), (16, 24), (24, 40), (40, 40)]
    pools = [False, True, False, True]
    h = 20
    st = B.F16 if storage == "f16" else B.F32
    layers, ws = [], []
    hh = h
    for i, (ci, co) in enumerate(chans):
        spec = synth.LayerSpec("s%d" % i, ci, co, hh, hh, 1, 1.0 if i == 0 else 0.5, sigma=None,
                               x_dist="uniform_01")
        w, b, _ = synth.gen_weights(spec, 900 + i)
        layers.append(B.Layer(w, synth.PATTERNS8, 1, st, b))
        ws.append((w, b))
        if pools[i]:
            hh //= 2
    x = synth.gen_input(synth.LayerSpec("in", 3, 16, h, h, 1, 1.0, x_dist="uniform_01"), 2, 901)
    stack = B.Stack(layers, pools, 2, h, h, B.RELU)
    xt = torch.from_numpy(x).cuda()
    xh = x
    if storage == "f16":
        xt = xt.half()
    y = torch.empty(stack.out_shape, dtype=xt.dtype, device="cuda")
    stack.forward(xt, y)
    torch.cuda.synchronize()
    a = xh
    for (w, b), pool in zip(ws, pools):
        a = oracle.conv3x3(a, w, b, 1, True, storage)
        if storage == "f16":        # activations are stored as fp16 between layers
            a = a.astype(np.float16).astype(np.float32)
        if pool:
            a = oracle.maxpool2x2(a)
    check_close(y.float().cpu().numpy(), a, storage, "stack")
    # host entry point gives the same result
    x_host = xt.cpu()
    y_host = torch.empty(stack.out_shape, dtype=xt.dtype)
    stack.forward_host(x_host, y_host)
    assert torch.equal(y_host, y.cpu()) or storage == "f32" and np.allclose(
        y_host.numpy(), y.cpu().numpy(), rtol=0, atol=1e-5)
    stack.close()


def test_stack_graph_replay_matches_the_eager_forward():
    chans = [(3, 16), (16, 32), (32, 32), (32, 48)]
    pools = [False, True, False, True]
    h = 24
    layers = []
    for i, (ci, co) in enumerate(chans):
        spec = synth.LayerSpec("g%d" % i, ci, co, h, h, 1, 1.0 if i == 0 else 0.5, sigma=None, x_dist="uniform_01")
        w, b, _ = synth.gen_weights(spec, 700 + i)
        layers.append(B.Layer(w, synth.PATTERNS8, 1, B.F32, b))
    stack = B.Stack(layers, pools, 1, h, h, B.RELU)
    x = torch.rand(1, 3, h, h, device="cuda")
    y_eager = torch.empty(stack.out_shape, device="cuda")
    y_graph = torch.zeros(stack.out_shape, device="cuda")
    stack.forward(x, y_eager)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with pytest.raises(B.PconvError):
        stack.replay(side)                      # nothing captured yet
    stack.capture(x, y_graph, side)
    for _ in range(3):                          # replays reuse the (zeroed) workspace correctly
        y_graph.zero_()
        side.synchronize()
        stack.replay(side)
        side.synchronize()
        assert torch.equal(y_graph, y_eager) or torch.allclose(y_graph, y_eager, rtol=1e-5, atol=1e-6)
    # the host entry point captures on its own buffers when the stream allows it
    xh = x.cpu().pin_memory()
    yh = torch.empty(stack.out_shape).pin_memory()
    for _ in range(2):
        stack.forward_host(xh, yh, side)
        assert torch.allclose(yh, y_eager.cpu(), rtol=1e-5, atol=1e-6)
    stack.forward_host(xh, yh)                  # default stream: eager path
    assert torch.allclose(yh, y_eager.cpu(), rtol=1e-5, atol=1e-6)
    assert B.pconv_device_status(layers[0].handle)[0] == 0
    stack.close()
