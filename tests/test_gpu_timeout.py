"""The give-up path of the tiled kernel, exercised without faulting or hanging anything.

Every wait in the kernel is bounded.  The development build of the library can make one producer
thread leave out its arrival for one chunk and shorten the bound: the consumers of that chunk
then run out of patience (a fraction of a millisecond), record the wait in the status word, skip
their remaining work and leave through the common exit, where the Tensor Memory columns are
handed back.  The tests check that the failure is reported (by pconv_device_status, by the host
entry point of a stack and by pconv_stack_status) and that the same GPU context computes correct
results right afterwards."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import check_close

pytestmark = pytest.mark.gpu

TIMEOUT = 10            # PCONV_ERR_DEVICE_TIMEOUT
SPIN_LIMIT = 2048       # tries of <= 200 ns each: a wait gives up after ~0.4 ms


@pytest.fixture(scope="module", autouse=True)
def dev_library():
    old = B.use_library(pbuild.build(dev=True))
    yield
    B.lib().pconv_dev_withhold(-1, 0)
    B.use_library(None)
    B._lib = old


def _arm(chunk):
    assert B.lib().pconv_dev_withhold(chunk, SPIN_LIMIT) == 0


def _disarm():
    assert B.lib().pconv_dev_withhold(-1, 0) == 0


def _case(c_in, c_out, h, n, seed, storage="f32"):
    spec = synth.LayerSpec("t", c_in, c_out, h, h, 1, 0.4)
    w, b, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    layer = B.Layer(w, synth.PATTERNS8, 1, B.F16 if storage == "f16" else B.F32, b)
    xt = torch.from_numpy(x).cuda()
    if storage == "f16":
        xt = xt.half()
    return layer, xt, oracle.conv3x3(x, w, b, 1, True, storage)


@pytest.mark.parametrize("storage", ["f32", "f16"])
def test_abandoned_wait_is_reported_and_the_gpu_stays_usable(storage):
    layer, x, ref = _case(32, 32, 14, 2, 5, storage)
    check_close(layer.forward(x).float().cpu().numpy(), ref, storage, "before")
    assert B.pconv_device_status(layer.handle) == (0, 0)
    _arm(1)
    layer.forward(x)
    torch.cuda.synchronize()
    status, where = B.pconv_device_status(layer.handle)
    assert status == TIMEOUT and where in (1, 2, 3), (status, where)
    _disarm()
    assert B.pconv_device_status(layer.handle)[0] == TIMEOUT          # sticky until cleared
    assert B.lib().pconv_dev_clear_status(layer.handle) == 0
    check_close(layer.forward(x).float().cpu().numpy(), ref, storage, "after the abandoned launch")
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


def test_abandoned_wait_in_the_channel_split_path_then_cleared_workspace():
    layer, x, ref = _case(128, 96, 28, 1, 31)
    assert B.pconv_plan(layer.handle, 1, 28, 28, 0, True)["channel_splits"] > 1
    check_close(layer.forward(x, split=True).cpu().numpy(), ref, "f32", "before")
    _arm(0)
    layer.forward(x, split=True)
    torch.cuda.synchronize()
    assert B.pconv_device_status(layer.handle)[0] == TIMEOUT
    _disarm()
    assert B.lib().pconv_dev_clear_status(layer.handle) == 0
    layer._ws.zero_()        # the contract: clear the workspace after an abandoned launch
    check_close(layer.forward(x, split=True).cpu().numpy(), ref, "f32", "after")
    assert not layer._ws.any()
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()


def test_chain_kernel_reports_an_abandoned_wait_and_recovers():
    """The same inside a chain (several layers in one persistent kernel): the layer whose chunk
    never arrives gives up, the grid-wide crossing still completes (every CTA counts itself in,
    finished or not), the launch ends, and after pconv_stack_status the stack works again."""
    specs = [synth.LayerSpec("a", 16, 32, 14, 14, 1, 0.5), synth.LayerSpec("b", 32, 32, 14, 14, 1, 0.5),
             synth.LayerSpec("c", 32, 16, 14, 14, 1, 0.5)]
    ws, layers = [], []
    for i, s in enumerate(specs):
        w, b, _ = synth.gen_weights(s, 60 + i)
        ws.append((w, b))
        layers.append(B.Layer(w, synth.PATTERNS8, 1, B.F32, b))
    x = synth.gen_input(specs[0], 1, 60)
    ref = x
    for w, b in ws:
        ref = oracle.conv3x3(ref, w, b, 1, True)
    stack = B.Stack(layers, [False] * 3, 1, 14, 14, B.RELU | B.CHAIN)
    assert stack.launches() == 1
    xt = torch.from_numpy(x).cuda()
    y = torch.empty(stack.out_shape, device="cuda")
    stack.forward(xt, y)
    torch.cuda.synchronize()
    check_close(y.cpu().numpy(), ref, "f32", "chain before")
    _arm(1)
    stack.forward(xt, y)
    torch.cuda.synchronize()
    _disarm()
    status, where = stack.status()
    assert status == TIMEOUT and where in (1, 2, 3, 9)
    assert stack.status() == (0, 0)
    y.fill_(float("nan"))
    stack.forward(xt, y)
    torch.cuda.synchronize()
    check_close(y.cpu().numpy(), ref, "f32", "chain after")
    stack.close()


def test_stack_host_entry_point_reports_the_abandoned_wait():
    specs = [synth.LayerSpec("a", 16, 32, 12, 12, 1, 0.5, pool_after=True),
             synth.LayerSpec("b", 32, 32, 6, 6, 1, 0.5)]
    ws, layers = [], []
    for i, s in enumerate(specs):
        w, b, _ = synth.gen_weights(s, 40 + i)
        ws.append((w, b))
        layers.append(B.Layer(w, synth.PATTERNS8, 1, B.F32, b))
    x = synth.gen_input(specs[0], 2, 40)
    ref = oracle.conv3x3(x, ws[0][0], ws[0][1], 1, True)
    ref = oracle.conv3x3(oracle.maxpool2x2(ref), ws[1][0], ws[1][1], 1, True)
    stack = B.Stack(layers, [True, False], 2, 12, 12, B.RELU)
    side = torch.cuda.Stream()
    y = np.empty(stack.out_shape, np.float32)
    stack.forward_host(x, y, side)
    check_close(y, ref, "f32", "stack before")
    assert stack.status() == (0, 0)
    _arm(1)
    with pytest.raises(B.PconvError) as e:
        stack.forward_host(x, y, side)
    assert e.value.status == TIMEOUT
    _disarm()
    status, where = stack.status()
    assert status == TIMEOUT and where in (1, 2, 3)
    assert stack.status() == (0, 0)                      # the call cleared the record
    y[:] = np.nan
    stack.forward_host(x, y, side)
    check_close(y, ref, "f32", "stack after")
    stack.close()
