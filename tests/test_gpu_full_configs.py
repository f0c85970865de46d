"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the GPU runs
the whole configuration; the oracle recomputes whole images for the stacks and a sample of
images for the large-batch layers."""
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


def test_config2_vgg16_stack_batch1_like_the_bench():
    cfg = synth.config(2)
    layers = _make_layers(cfg)
    s0 = cfg.layers[0]
    x = synth.gen_input(s0, 1, synth.layer_seed(2, 0))
    stack = B.Stack([l[3] for l in layers], [l[0].pool_after for l in layers], 1, s0.h, s0.w, B.RELU)
    y = torch.empty(stack.out_shape, device="cuda")
    stack.forward(torch.from_numpy(x).cuda(), y)
    torch.cuda.synchronize()
    ref = _oracle_chain(layers, x, "f32")
    check_close(y.cpu().numpy(), ref, "f32", "VGG-16 stack")
    # every layer alone on a fresh input of the config's distribution (binding check)
    for li, (spec, w, b, layer) in enumerate(layers):
        xi = synth.gen_input(spec, 1, synth.layer_seed(2, li))
        got = layer.forward(torch.from_numpy(xi).cuda(), relu=True, split=True)
        torch.cuda.synchronize()
        check_close(got.cpu().numpy(), oracle.conv3x3(xi, w, b, 1, True), "f32", spec.name)
    stack.close()


def test_config4_cifar_stack_fp16_batch256_sampled_images():
    cfg = synth.config(4)
    layers = _make_layers(cfg)
    s0 = cfg.layers[0]
    x = synth.gen_input(s0, cfg.batch, synth.layer_seed(4, 0))
    stack = B.Stack([l[3] for l in layers], [l[0].pool_after for l in layers], cfg.batch, s0.h,
                    s0.w, B.RELU)
    y = torch.empty(stack.out_shape, dtype=torch.float16, device="cuda")
    stack.forward(torch.from_numpy(x).cuda().half(), y)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy()
    for n in (0, 101, 255):
        ref = _oracle_chain(layers, x[n:n + 1], "f16")
        check_close(got[n:n + 1], ref, "f16", "CIFAR stack image %d" % n)
    # the binding check: single layers on fresh inputs, three of them across the depth
    for li in (1, 6, 12):
        spec, w, b, layer = layers[li]
        xi = synth.gen_input(spec, 8, synth.layer_seed(4, li))
        g = layer.forward(torch.from_numpy(xi).cuda().half(), relu=True)
        torch.cuda.synchronize()
        check_close(g.float().cpu().numpy(), oracle.conv3x3(xi, w, b, 1, True, "f16"), "f16", spec.name)
    stack.close()


@pytest.mark.parametrize("li", [0, 3, 7, 13, 15])
def test_config3_resnet_layers_batch32_sampled_images(li):
    cfg = synth.config(3, 32)
    spec = cfg.layers[li]
    w, b, _ = synth.gen_weights(spec, synth.layer_seed(3, li), cfg.patterns)
    x = synth.gen_input(spec, 32, synth.layer_seed(3, li))
    layer = B.Layer(w, cfg.patterns, spec.stride, B.F32, b, strict4=True)
    got = layer.forward(torch.from_numpy(x).cuda(), relu=True, split=True)
    torch.cuda.synchronize()
    got = got.cpu().numpy()
    for n in (0, 17, 31):
        check_close(got[n:n + 1], oracle.conv3x3(x[n:n + 1], w, b, spec.stride, True), "f32",
                    "%s image %d" % (spec.name, n))
    layer.close()


@pytest.mark.parametrize("li", [0, 1])
def test_config5_imbalance_layers_batch64_sampled_images(li):
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
    torch.cuda.synchronize()
    got = got.cpu().numpy()
    for n in (0, 63):
        check_close(got[n:n + 1], oracle.conv3x3(x[n:n + 1], w, b, spec.stride, True), "f32",
                    "%s image %d" % (spec.name, n))
    layer.close()
