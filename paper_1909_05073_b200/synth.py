"""Seeded synthetic workloads for the PCONV forward pass (inputs only: no convolution
arithmetic lives here, so the CUDA library's tests and the CPU oracle can both draw from it).

The layer shapes stand in for the paper's evaluation models (VGG-16 and ResNet-50 on ImageNet
and CIFAR-10, "Experimental Results" section): timing and parity depend only on shapes and on the
sparsity structure, so weights are random draws carrying the two PCONV sparsities -- each kept
(filter, input-channel) kernel has exactly 4 non-zeros in one pattern of the set (pattern pruning,
2.25x = 9/4), and whole kernels are zeroed with probability 1 - keep (connectivity pruning).

Pattern masks are 9-bit integers, bit 3*u+v for kernel row u and column v (centre = bit 4).
Ids 0-3 are the four designed SCPs (centre plus three of the four edge neighbours, in the order
the paper lists them: without down, without right, without up, without left); ids 4-7 are this
build's choice for the paper's unspecified "random patterns with 4 non-zero elements": the four
2x2 blocks that contain the centre.
"""
from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

SEED0 = 190905073

SCP4 = (0x03A, 0x09A, 0x0B8, 0x0B2)
PATTERNS8 = SCP4 + (0x01B, 0x036, 0x0D8, 0x1B0)
# four further arbitrary 4-tap masks (two of them without the centre) for the 12-pattern sweep
PATTERNS12 = PATTERNS8 + (0x055, 0x0AA, 0x113, 0x18C)

UNIFORM8 = (0.125,) * 8
SKEWED8 = (0.3, 0.2, 0.15, 0.1, 0.1, 0.05, 0.05, 0.05)


def mask_array(mask: int) -> np.ndarray:
    """3x3 {0,1} array of a 9-bit mask."""
    return np.array([(mask >> b) & 1 for b in range(9)], dtype=np.float32).reshape(3, 3)


@dataclass(frozen=True)
class LayerSpec:
    name: str
    c_in: int
    c_out: int
    h: int                      # input height
    w: int                      # input width
    stride: int = 1
    keep: float = 0.5           # kernel keep probability; < 0 means per-filter U(0.1, 0.9)
    probs: Tuple[float, ...] = UNIFORM8
    sigma: Optional[float] = 0.05   # None = He-normal on the dense fan-in 9*c_in
    x_dist: str = "uniform_pm1"     # uniform_pm1 | uniform_01 | relu_normal
    pool_after: bool = False        # 2x2 max-pool follows this layer (stacks only)

    @property
    def h_out(self):
        return (self.h - 1) // self.stride + 1

    @property
    def w_out(self):
        return (self.w - 1) // self.stride + 1


@dataclass(frozen=True)
class Config:
    cid: int
    name: str
    layers: Tuple[LayerSpec, ...]
    batch: int
    storage: str = "f32"        # "f32" | "f16" (weights/activations fp16, accumulate fp32)
    chained: bool = False       # True: layer k+1 consumes layer k's output (a stack)
    patterns: Tuple[int, ...] = PATTERNS8


_VGG = [(3, 64), (64, 64), "P", (64, 128), (128, 128), "P", (128, 256), (256, 256), (256, 256),
        "P", (256, 512), (512, 512), (512, 512), "P", (512, 512), (512, 512), (512, 512)]


def _vgg_layers(size, keep_first, keep_rest, sigma, x_dist):
    layers, h, idx = [], size, 0
    for item in _VGG:
        if item == "P":
            layers[-1] = replace(layers[-1], pool_after=True)
            h //= 2
            continue
        idx += 1
        layers.append(LayerSpec("conv%d" % idx, item[0], item[1], h, h, 1,
                                keep_first if idx == 1 else keep_rest, UNIFORM8, sigma, x_dist))
    return tuple(layers)


def _resnet_layers():
    out = []
    plan = [(64, 56, 3, False), (128, 28, 4, True), (256, 14, 6, True), (512, 7, 3, True)]
    for si, (c, hw, blocks, down) in enumerate(plan, start=1):
        for b in range(1, blocks + 1):
            s = 2 if (down and b == 1) else 1
            h_in = hw * s
            out.append(LayerSpec("stage%d_b%d" % (si, b), c, c, h_in, h_in, s, 0.35, SKEWED8,
                                 None, "relu_normal"))
    return tuple(out)


def config(cid: int, batch: Optional[int] = None) -> Config:
    """The five benchmark configurations (1-based ids)."""
    if cid == 1:
        return Config(1, "single 64->64 56x56",
                      (LayerSpec("c1", 64, 64, 56, 56, 1, 0.5),), batch or 1)
    if cid == 2:
        return Config(2, "VGG-16 conv stack 224x224",
                      _vgg_layers(224, 1.0, 0.3, None, "uniform_01"), batch or 1, chained=True)
    if cid == 3:
        return Config(3, "ResNet-50 3x3 bottleneck convs", _resnet_layers(), batch or 1)
    if cid == 4:
        return Config(4, "CIFAR-shaped VGG-16 32x32 fp16 storage",
                      _vgg_layers(32, 0.25, 0.25, 0.05, "uniform_pm1"), batch or 256,
                      storage="f16", chained=True)
    if cid == 5:
        return Config(5, "load-imbalance stress 512->512",
                      (LayerSpec("s1", 512, 512, 14, 14, 1, -1.0),
                       LayerSpec("s2", 512, 512, 28, 28, 2, -1.0)), batch or 64)
    raise ValueError("config id must be 1..5")


def layer_seed(cid: int, layer_index: int) -> int:
    return SEED0 + 1000 * cid + layer_index


def gen_weights(spec: LayerSpec, seed: int, patterns=PATTERNS8):
    """Dense OIHW fp32 weights with the PCONV zeros in place, fp32 bias, per-kernel pattern ids
    (-1 = pruned).  Draw order: weights, keep mask, pattern ids, (masking), bias."""
    rng = np.random.default_rng(seed)
    sigma = spec.sigma if spec.sigma is not None else float(np.sqrt(2.0 / (9 * spec.c_in)))
    w = rng.normal(0.0, sigma, (spec.c_out, spec.c_in, 3, 3)).astype(np.float32)
    if spec.keep < 0:
        r = rng.uniform(0.1, 0.9, spec.c_out)
        kept = rng.random((spec.c_out, spec.c_in)) < r[:, None]
    else:
        kept = rng.random((spec.c_out, spec.c_in)) < spec.keep
    n_pat = len(patterns)
    probs = np.asarray(spec.probs[:n_pat], dtype=np.float64)
    if len(probs) < n_pat:
        probs = np.full(n_pat, 1.0 / n_pat)
    probs = probs / probs.sum()
    ids = rng.choice(n_pat, p=probs, size=(spec.c_out, spec.c_in))
    masks = np.stack([mask_array(m) for m in patterns])          # [n_pat,3,3]
    w *= masks[ids]
    w *= kept[:, :, None, None]
    bias = rng.normal(0.0, 0.01, spec.c_out).astype(np.float32)
    ids = np.where(kept, ids, -1).astype(np.int8)
    return w, bias, ids


def gen_input(spec: LayerSpec, batch: int, seed: int) -> np.ndarray:
    """fp32 NCHW input of the layer's distribution (seeded separately from the weights)."""
    rng = np.random.default_rng(seed + 500)
    shape = (batch, spec.c_in, spec.h, spec.w)
    if spec.x_dist == "uniform_pm1":
        return rng.uniform(-1.0, 1.0, shape).astype(np.float32)
    if spec.x_dist == "uniform_01":
        return rng.uniform(0.0, 1.0, shape).astype(np.float32)
    if spec.x_dist == "relu_normal":
        return np.maximum(rng.normal(0.0, 1.0, shape), 0.0).astype(np.float32)
    raise ValueError(spec.x_dist)
