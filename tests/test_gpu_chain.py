"""Chains: with PCONV_CHAIN a stack runs consecutive layers whose launch plans are single waves of
CTAs (batch-1 inference) as ONE persistent kernel -- Tensor Memory and the CTAs stay, layers are
crossed on a grid-wide count.  The result must be the oracle's, the same as with one launch per
layer (the default), and the counters must be back at zero so that the next forward works."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import Guarded, check_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()
    B.lib()


def _stack_case(specs, n, storage, seed):
    st = B.F16 if storage == "f16" else B.F32
    ws, layers = [], []
    for i, s in enumerate(specs):
        w, b, _ = synth.gen_weights(s, seed + i)
        ws.append((w, b))
        layers.append(B.Layer(w, synth.PATTERNS8, 1, st, b))
    x = synth.gen_input(specs[0], n, seed)
    a = x
    for (w, b), s in zip(ws, specs):
        a = oracle.conv3x3(a, w, b, 1, True, storage)
        if storage == "f16":
            a = a.astype(np.float16).astype(np.float32)
        if s.pool_after:
            a = oracle.maxpool2x2(a)
    return layers, x, a


CASES = [
    # (layer specs as (c_in, c_out, h, pool_after), batch, storage)
    ([(16, 32, 14, False), (32, 32, 14, False), (32, 48, 14, False)], 1, "f32"),
    ([(8, 16, 28, True), (16, 64, 14, False), (64, 64, 14, True), (64, 32, 7, False)], 1, "f32"),
    ([(64, 128, 14, False), (128, 128, 14, False)], 2, "f32"),           # channel split in both layers
    ([(24, 40, 12, False), (40, 40, 12, True), (40, 16, 6, False)], 1, "f16"),
    ([(3, 16, 40, False), (16, 16, 40, True), (16, 32, 20, False), (32, 32, 20, False)], 1, "f32"),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "%dlayers-n%d-%s" % (len(c[0]), c[1], c[2]))
def test_chain_matches_the_oracle_and_the_layer_by_layer_stack(case):
    shapes, n, storage = case
    specs = [synth.LayerSpec("l%d" % i, ci, co, h, h, 1, 0.4, pool_after=p) for i, (ci, co, h, p) in enumerate(shapes)]
    layers, x, ref = _stack_case(specs, n, storage, 3100 + len(shapes) + shapes[0][0])
    pools = [s.pool_after for s in specs]
    dt = torch.float16 if storage == "f16" else torch.float32
    xt = torch.from_numpy(x).cuda().to(dt)
    chained = B.Stack(layers, pools, n, specs[0].h, specs[0].w, B.RELU | B.CHAIN)
    plain = B.Stack(layers, pools, n, specs[0].h, specs[0].w, B.RELU)
    assert plain.launches() == len(specs)
    assert chained.launches() < len(specs), "no chain was formed for a batch-1 stack of small layers"
    for rep in range(3):                      # the counters must come back to zero every time
        y = Guarded(chained.out_shape, dt, fill=float("nan"))
        chained.forward(xt, y.t)
        y.check("chain output")
        check_close(y.t.float().cpu().numpy(), ref, storage, "chain, forward %d" % rep)
    y2 = torch.empty(plain.out_shape, dtype=dt, device="cuda")
    plain.forward(xt, y2)
    torch.cuda.synchronize()
    check_close(y2.float().cpu().numpy(), ref, storage, "layer by layer")
    assert chained.status() == (0, 0) and plain.status() == (0, 0)
    chained.close()
    plain.close()


def test_chain_inside_a_captured_graph_and_through_the_host_entry_point():
    specs = [synth.LayerSpec("a", 16, 32, 14, 14, 1, 0.4), synth.LayerSpec("b", 32, 32, 14, 14, 1, 0.4)]
    layers, x, ref = _stack_case(specs, 1, "f32", 77)
    stack = B.Stack(layers, [False, False], 1, 14, 14, B.RELU | B.CHAIN)
    assert stack.launches() == 1
    side = torch.cuda.Stream()
    y = np.empty(stack.out_shape, np.float32)
    for _ in range(3):
        y[:] = np.nan
        stack.forward_host(x, y, side)      # replays its device part from a captured graph
        check_close(y, ref, "f32", "chain through the host entry point")
    assert stack.status() == (0, 0)
    stack.close()
