"""Seeded synthetic convolution workloads.

This module holds layer shapes and random-number recipes only — none of the
method's arithmetic — so that the tests can hand the very same arrays to the
CUDA path and to the CPU oracle.  The layers are shaped like the CNNs the
paper evaluates (ResNet-18 and MobileNet-v1 on one 224 x 224 image, Section 4.2);
trained weights and images are replaced by draws from NumPy's PCG64 generator.

Seed of a layer = 1000 * config + index of the layer in the config, + 500 for
the large-batch variant of the config.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class ConvLayer:
    name: str
    N: int
    Cin: int
    Cout: int
    H: int
    W: int
    k: int
    stride: int = 1
    pad: int = 0
    dilation: int = 1
    groups: int = 1
    relu: bool = True
    x_dist: str = "relu_normal"    # "relu_normal" | "normal" | "uniform"
    w_dist: str = "kaiming"        # "kaiming" | "normal" | "uniform"
    bias_dist: str = "normal0.1"   # "normal0.1" | "zero"
    seed: int = 0

    @property
    def OH(self) -> int:
        return (self.H + 2 * self.pad - self.dilation * (self.k - 1) - 1) // self.stride + 1

    @property
    def OW(self) -> int:
        return (self.W + 2 * self.pad - self.dilation * (self.k - 1) - 1) // self.stride + 1

    @property
    def direct_flops(self) -> int:
        """Multiply-adds x 2 of the plain definition (the metric's numerator)."""
        return 2 * self.N * self.Cout * (self.Cin // self.groups) * self.OH * self.OW * self.k * self.k

    def with_batch(self, N: int, seed_offset: int = 0) -> "ConvLayer":
        return replace(self, N=N, seed=self.seed + seed_offset)


def make_inputs(layer: ConvLayer):
    """(x, w, bias) as fp32 NumPy arrays; bias is None when the recipe says zero."""
    rng = np.random.Generator(np.random.PCG64(layer.seed))
    xs = (layer.N, layer.Cin, layer.H, layer.W)
    cpg = layer.Cin // layer.groups
    ws = (layer.Cout, cpg, layer.k, layer.k)
    if layer.x_dist == "uniform":
        x = rng.uniform(-1.0, 1.0, size=xs).astype(np.float32)
    elif layer.x_dist == "normal":
        x = rng.standard_normal(size=xs, dtype=np.float32)
    elif layer.x_dist == "relu_normal":
        x = np.maximum(rng.standard_normal(size=xs, dtype=np.float32), np.float32(0))
    else:
        raise ValueError(layer.x_dist)
    if layer.w_dist == "uniform":
        w = rng.uniform(-1.0, 1.0, size=ws).astype(np.float32)
    elif layer.w_dist == "normal":
        w = rng.standard_normal(size=ws, dtype=np.float32)
    elif layer.w_dist == "kaiming":
        fan_in = cpg * layer.k * layer.k
        w = (rng.standard_normal(size=ws, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))).astype(np.float32)
    else:
        raise ValueError(layer.w_dist)
    if layer.bias_dist == "zero":
        bias = None
    elif layer.bias_dist == "normal0.1":
        bias = (rng.standard_normal(size=(layer.Cout,), dtype=np.float32) * np.float32(0.1)).astype(np.float32)
    else:
        raise ValueError(layer.bias_dist)
    return x, w, bias


def integer_inputs(layer: ConvLayer, lo: int = -4, hi: int = 4):
    """Small-integer-valued fp32 tensors of the layer's shape: every product and
    partial sum is exactly representable, so any correct evaluation order gives
    bit-identical results."""
    rng = np.random.Generator(np.random.PCG64(layer.seed + 77))
    x = rng.integers(lo, hi + 1, size=(layer.N, layer.Cin, layer.H, layer.W)).astype(np.float32)
    w = rng.integers(lo, hi + 1, size=(layer.Cout, layer.Cin // layer.groups, layer.k, layer.k)).astype(np.float32)
    bias = rng.integers(lo, hi + 1, size=(layer.Cout,)).astype(np.float32)
    return x, w, bias


# ---------------------------------------------------------------------------
# The five configurations.
# ---------------------------------------------------------------------------
def config0():
    """One 3x3 conv, N=1, 32->32, 28x28, uniform[-1,1], bias zero."""
    return [ConvLayer("c0_3x3_32_28", 1, 32, 32, 28, 28, 3, 1, 1, relu=False, x_dist="uniform",
                      w_dist="uniform", bias_dist="zero", seed=0)]


def config1(batch: int = 1):
    """ResNet-18-style 3x3 stride-1 pad-1 layers, Cin = Cout."""
    off = 0 if batch == 1 else 500
    shapes = [(64, 56), (128, 28), (256, 14), (512, 7)]
    return [ConvLayer("c1_3x3_%d_%d" % (c, h), batch, c, c, h, h, 3, 1, 1, seed=1000 + i + off)
            for i, (c, h) in enumerate(shapes)]


def config2(batch: int = 1):
    """Every conv of a ResNet-18 forward on 3 x 224 x 224 (BN folded into weights and bias)."""
    off = 0 if batch == 1 else 500
    layers = [("stem_7x7s2", 3, 64, 224, 7, 2, 3)]
    for i in range(4):
        layers.append(("l1_3x3_%d" % i, 64, 64, 56, 3, 1, 1))
    cin, res = 64, 56
    for stage, c in ((2, 128), (3, 256), (4, 512)):
        layers.append(("l%d_3x3s2" % stage, cin, c, res, 3, 2, 1))
        layers.append(("l%d_down1x1s2" % stage, cin, c, res, 1, 2, 0))
        res //= 2
        for i in range(3):
            layers.append(("l%d_3x3_%d" % (stage, i), c, c, res, 3, 1, 1))
        cin = c
    out = []
    for i, (name, ci, co, h, k, s, p) in enumerate(layers):
        relu = "down" not in name
        out.append(ConvLayer("c2_" + name, batch, ci, co, h, h, k, s, p, relu=relu, seed=2000 + i + off))
    return out


def config3(batch: int = 1):
    """MobileNet-v1 (width 1.0, 224 x 224): conv1, then 13 x (depthwise 3x3, pointwise 1x1)."""
    off = 0 if batch == 1 else 500
    out = [ConvLayer("c3_conv1_3x3s2", batch, 3, 32, 224, 224, 3, 2, 1, seed=3000 + off)]
    plan = [(32, 64, 1), (64, 128, 2), (128, 128, 1), (128, 256, 2), (256, 256, 1), (256, 512, 2),
            (512, 512, 1), (512, 512, 1), (512, 512, 1), (512, 512, 1), (512, 512, 1),
            (512, 1024, 2), (1024, 1024, 1)]
    res, idx = 112, 1
    for j, (ci, co, s) in enumerate(plan):
        out.append(ConvLayer("c3_dw%d_3x3s%d" % (j + 1, s), batch, ci, ci, res, res, 3, s, 1, groups=ci,
                             seed=3000 + idx + off))
        idx += 1
        res = (res + 2 - 3) // s + 1
        out.append(ConvLayer("c3_pw%d_1x1" % (j + 1), batch, ci, co, res, res, 1, 1, 0, seed=3000 + idx + off))
        idx += 1
    return out


def config4(batch: int = 64):
    """Large-batch Winograd stress shapes, N(0,1) data, bias zero, no ReLU."""
    shapes = [("3x3_256_56", 256, 56, 3, 1), ("3x3_512_56", 512, 56, 3, 1),
              ("5x5_128_28", 128, 28, 5, 2), ("7x7_128_28", 128, 28, 7, 3)]
    return [ConvLayer("c4_" + name, batch, c, c, h, h, k, 1, p, relu=False, x_dist="normal", w_dist="normal",
                      bias_dist="zero", seed=4000 + i)
            for i, (name, c, h, k, p) in enumerate(shapes)]
