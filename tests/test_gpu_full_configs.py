"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the GPU runs
each whole configuration and the oracle recomputes every image of it (the sub-tile table of a CTA
depends on the image index, so a sampled image proves nothing about its neighbours).

Deep in a chained stack the activations shrink until the tolerance passes anything; the binding
check is therefore every layer alone on a fresh input of the configuration's distribution, with
the scale-aware error bound of util.check_close."""
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


def _make_layers(cfg):
    st = B.F16 if cfg.storage == "f16" else B.F32
    out = []
    for li, spec in enumerate(cfg.layers):
        w, b, _ = synth.gen_weights(spec, synth.layer_seed(cfg.cid, li), cfg.patterns)
        out.append((spec, w, b, B.Layer(w, cfg.patterns, spec.stride, st, b, strict4=True)))
    return out


def _oracle_chain(layers, x, storage):
    a = x
    for spec, w, b, _ in layers:
        a = oracle.conv3x3(a, w, b, spec.stride, True, storage)
        if storage == "f16":
            a = a.astype(np.float16).astype(np.float32)
        if spec.pool_after:
            a = oracle.maxpool2x2(a)
    return a


def _status_ok(layer):
    status, where = B.pconv_device_status(layer.handle)
    assert status == 0, ("device status", status, where)


def test_config1_single_layer_batch1():
    cfg = synth.config(1)
    spec = cfg.layers[0]
    w, b, _ = synth.gen_weights(spec, synth.layer_seed(1, 0), cfg.patterns)
    x = synth.gen_input(spec, 1, synth.layer_seed(1, 0))
    layer = B.Layer(w, cfg.patterns, 1, B.F32, b, strict4=True)
    for split in (False, True):
        got = layer.forward(torch.from_numpy(x).cuda(), relu=True, split=split)
        check_close(got.cpu().numpy(), oracle.conv3x3(x, w, b, 1, True), "f32", "config 1 split=%s" % split)
    _status_ok(layer)
    layer.close()


def test_config2_vgg16_stack_batch1_like_the_bench():
    cfg = synth.config(2)
    layers = _make_layers(cfg)
    s0 = cfg.layers[0]
    x = synth.gen_input(s0, 1, synth.layer_seed(2, 0))
    stack = B.Stack([l[3] for l in layers], [l[0].pool_after for l in layers], 1, s0.h, s0.w, B.RELU)
    y = Guarded(stack.out_shape, torch.float32, fill=float("nan"))
    stack.forward(torch.from_numpy(x).cuda(), y.t)
    y.check("VGG-16 stack output")
    ref = _oracle_chain(layers, x, "f32")
    check_close(y.t.cpu().numpy(), ref, "f32", "VGG-16 stack")
    # every layer alone on a fresh input of the config's distribution (binding check), as the
    # stack launches it: with the channel-split workspace, and with the fused pool where one follows
    for li, (spec, w, b, layer) in enumerate(layers):
        xi = synth.gen_input(spec, 1, synth.layer_seed(2, li))
        ref_i = oracle.conv3x3(xi, w, b, 1, True)
        got = layer.forward(torch.from_numpy(xi).cuda(), relu=True, split=True)
        check_close(got.cpu().numpy(), ref_i, "f32", spec.name)
        if spec.pool_after:
            got = layer.forward(torch.from_numpy(xi).cuda(), relu=True, split=True, pool=True)
            check_close(got.cpu().numpy(), oracle.maxpool2x2(ref_i), "f32", spec.name + " pooled")
        _status_ok(layer)
    stack.close()


def test_config4_cifar_stack_fp16_batch256_every_image():
    cfg = synth.config(4)
    layers = _make_layers(cfg)
    s0 = cfg.layers[0]
    x = synth.gen_input(s0, cfg.batch, synth.layer_seed(4, 0))
    stack = B.Stack([l[3] for l in layers], [l[0].pool_after for l in layers], cfg.batch, s0.h,
                    s0.w, B.RELU)
    y = Guarded(stack.out_shape, torch.float16, fill=float("nan"))
    stack.forward(torch.from_numpy(x).cuda().half(), y.t)
    y.check("CIFAR stack output")
    got = y.t.float().cpu().numpy()
    ref = _oracle_chain(layers, x, "f16")
    check_close(got, ref, "f16", "CIFAR stack, all %d images" % cfg.batch)
    stack.close()


@pytest.mark.parametrize("li", range(13))
def test_config4_single_layers_fp16_batch256_every_image(li):
    """The binding check of config 4: each of the 13 layers alone at the full batch, on a fresh
    input of the config's distribution -- the first layer (many filters without any kernel at
    keep 0.25) and the 2x2 maps included."""
    cfg = synth.config(4)
    spec = cfg.layers[li]
    w, b, ids = synth.gen_weights(spec, synth.layer_seed(4, li), cfg.patterns)
    if li == 0:
        assert ((ids >= 0).sum(1) == 0).any()      # filters with no surviving kernel exist
    x = synth.gen_input(spec, cfg.batch, synth.layer_seed(4, li))
    layer = B.Layer(w, cfg.patterns, 1, B.F16, b, strict4=True)
    ref = oracle.conv3x3(x, w, b, 1, True, "f16")
    xt = torch.from_numpy(x).cuda().half()
    got = layer.forward(xt, relu=True, split=True)
    check_close(got.float().cpu().numpy(), ref, "f16", spec.name)
    if spec.pool_after:
        got = layer.forward(xt, relu=True, split=True, pool=True)
        check_close(got.float().cpu().numpy(), oracle.maxpool2x2(ref), "f16", spec.name + " pooled")
    _status_ok(layer)
    layer.close()


@pytest.mark.parametrize("batch", [1, 32])
@pytest.mark.parametrize("li", range(16))
def test_config3_resnet_layers_every_image(li, batch):
    cfg = synth.config(3, batch)
    spec = cfg.layers[li]
    w, b, _ = synth.gen_weights(spec, synth.layer_seed(3, li), cfg.patterns)
    x = synth.gen_input(spec, batch, synth.layer_seed(3, li))
    layer = B.Layer(w, cfg.patterns, spec.stride, B.F32, b, strict4=True)
    got = layer.forward(torch.from_numpy(x).cuda(), relu=True, split=True)
    check_close(got.cpu().numpy(), oracle.conv3x3(x, w, b, spec.stride, True), "f32",
                "%s batch %d" % (spec.name, batch))
    _status_ok(layer)
    layer.close()


@pytest.mark.parametrize("li", [0, 1])
def test_config5_imbalance_layers_batch64_every_image(li):
    cfg = synth.config(5)
    spec = cfg.layers[li]
    w, b, ids = synth.gen_weights(spec, synth.layer_seed(5, li), cfg.patterns)
    per = (ids >= 0).sum(1)
    assert per.min() < 100 and per.max() > 400          # the imbalance the config is about
    x = synth.gen_input(spec, cfg.batch, synth.layer_seed(5, li))
    layer = B.Layer(w, cfg.patterns, spec.stride, B.F32, b, strict4=True)
    s = layer.stats()
    assert s.max_group_kernels - s.min_group_kernels <= 0.02 * s.max_group_kernels
    got = layer.forward(torch.from_numpy(x).cuda(), relu=True)
    check_close(got.cpu().numpy(), oracle.conv3x3(x, w, b, spec.stride, True), "f32", spec.name)
    _status_ok(layer)
    layer.close()
