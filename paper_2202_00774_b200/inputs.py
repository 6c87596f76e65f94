"""Seeded synthetic inputs for SDGP tests and benchmarks.

This module only draws random tensors and describes workload shapes; it holds
none of the pruning or contraction arithmetic. Everything is numpy on the
host; bf16 tensors are returned as ``uint16`` bit patterns (row-major) so the
same bits can be handed to any consumer.

Workloads (synthetic stand-ins for the gradients and weights of the paper's
CIFAR-10 / ImageNet training runs, Section 4):
  * ``fc_small``       one fully connected layer, dO [256, 512], W [512, 256]
  * ``resnet9``        3x3 stride-1 pad-1 convolution layers of a 9-layer ResNet at batch 512
  * ``resnet50``       1x1 / 3x3 bottleneck convolutions of ResNet-50 at batch 256
  * ``gemm_large``     dO [16384, 4096], W [4096, 4096]
  * ``resnet18``       3x3 / stride-2 / shortcut convolutions of ResNet-18 (parity shapes)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even) and return the bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to IEEE binary16 (nearest, ties to even; numpy's conversion) and return the bit patterns."""
    with np.errstate(over="ignore"):
        return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def f16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(b, dtype=np.uint16).view(np.float16).astype(np.float32)


def bf16_bits_as_f16_bits(b: np.ndarray) -> np.ndarray:
    """The values of a bf16 tensor re-encoded as binary16 (rounded; the same draw in the other format)."""
    return f32_to_f16_bits(bf16_bits_to_f32(b))


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def normal_bf16(shape, std: float, seed: int, stream: int = 0) -> np.ndarray:
    """N(0, std^2) rounded to bf16."""
    g = _rng(seed, stream)
    return f32_to_bf16_bits(g.standard_normal(shape, dtype=np.float32) * np.float32(std))


def relu_masked_laplace_bf16(shape, seed: int, stream: int = 0, zero_fraction: float = 0.5) -> np.ndarray:
    """Laplace(0, 1) values with a Bernoulli(zero_fraction) share forced to exact +0.0,
    as a gradient that has passed back through a ReLU would look (Section 3.3 reports a
    large share of exact zeros in real data gradients)."""
    g = _rng(seed, stream)
    n = int(np.prod(shape))
    out = np.empty(n, np.uint16)
    step = 1 << 24
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        v = g.laplace(0.0, 1.0, hi - lo).astype(np.float32)
        v[g.random(hi - lo, dtype=np.float32) < zero_fraction] = 0.0
        out[lo:hi] = f32_to_bf16_bits(v)
    return out.reshape(shape)


def adversarial_groups_bf16(rows: int, K: int, seed: int) -> np.ndarray:
    """Rows full of ranking edge cases: ties, signed zeros, infinities, NaNs, denormals."""
    g = _rng(seed, 99)
    pool = np.array([0x0000, 0x8000, 0x3F80, 0xBF80, 0x3F80, 0x4000, 0xC000, 0x7F80, 0xFF80,
                     0x7FC0, 0xFFC1, 0x0001, 0x8001, 0x007F, 0x7F7F, 0xFF7F, 0x3F81, 0xBF81],
                    dtype=np.uint16)
    return pool[g.integers(0, pool.size, size=(rows, K))]


# ------------------------------------------------------------------ shapes


@dataclass(frozen=True)
class ConvLayer:
    name: str
    B: int
    H: int      # input (dD) height
    W: int      # input (dD) width
    Cin: int
    Cout: int
    R: int
    S: int
    stride: int
    pad: int
    groups: int = 1   # grouped convolution: W is [Cout, R, S, Cin / groups]

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def dense_macs(self) -> int:
        """True multiply-accumulates of the dense data-gradient contraction."""
        return self.B * self.P * self.Q * self.Cout * self.R * self.S * (self.Cin // self.groups)

    def dO_shape(self):
        return (self.B, self.P, self.Q, self.Cout)

    def W_shape(self):
        return (self.Cout, self.R, self.S, self.Cin // self.groups)

    def dD_shape(self):
        return (self.B, self.H, self.W, self.Cin)


def resnet9_layers(batch: int = 512) -> List[ConvLayer]:
    """3x3, stride 1, pad 1 layers (Cin -> Cout @ HxW) of the CIFAR-sized 9-layer ResNet."""
    spec = [(64, 128, 32), (128, 128, 16), (128, 128, 16), (128, 256, 16), (256, 512, 8),
            (512, 512, 4), (512, 512, 4)]
    return [ConvLayer("r9_%d_%dto%d_at%d" % (i, ci, co, hw), batch, hw, hw, ci, co, 3, 3, 1, 1)
            for i, (ci, co, hw) in enumerate(spec)]


def resnet50_stride1_layers(batch: int = 256) -> List[ConvLayer]:
    """Distinct stride-1 1x1 / 3x3 bottleneck convolutions of ResNet-50 (stages 1-4)."""
    out = []
    for stage, (hw, mid) in enumerate([(56, 64), (28, 128), (14, 256), (7, 512)], start=1):
        wide = 4 * mid
        out.append(ConvLayer("r50_s%d_1x1_%dto%d" % (stage, wide, mid), batch, hw, hw, wide, mid, 1, 1, 1, 0))
        out.append(ConvLayer("r50_s%d_3x3_%dto%d" % (stage, mid, mid), batch, hw, hw, mid, mid, 3, 3, 1, 1))
        out.append(ConvLayer("r50_s%d_1x1_%dto%d" % (stage, mid, wide), batch, hw, hw, mid, wide, 1, 1, 1, 0))
    out.insert(0, ConvLayer("r50_s1_1x1_64to64", batch, 56, 56, 64, 64, 1, 1, 1, 0))
    return out


def resnet50_layers(batch: int = 256):
    """Every distinct 1x1 / 3x3 convolution of the ResNet-50 bottleneck stages 1-4 with the number
    of times the network holds it: (layer, count) pairs. The stride-2 transitions sit on the 3x3
    convolution of each stage's first block and on its 1x1 projection shortcut."""
    out = []
    prev_wide = 64   # channels that enter stage 1 (from the stem)
    for stage, (hw, mid, blocks) in enumerate([(56, 64, 3), (28, 128, 4), (14, 256, 6), (7, 512, 3)], start=1):
        wide = 4 * mid
        s = 1 if stage == 1 else 2
        hin = hw * s   # spatial size entering the stage
        tag = "r50_s%d_" % stage
        # first block: reduce at the incoming size, 3x3 carries the stride, projection shortcut
        out.append((ConvLayer(tag + "1x1_%dto%d_at%d" % (prev_wide, mid, hin), batch, hin, hin, prev_wide, mid, 1, 1, 1, 0), 1))
        if s == 2:
            out.append((ConvLayer(tag + "3x3s2_%dto%d_at%d" % (mid, mid, hin), batch, hin, hin, mid, mid, 3, 3, 2, 1), 1))
        out.append((ConvLayer(tag + "proj%s_%dto%d_at%d" % ("s2" if s == 2 else "", prev_wide, wide, hin), batch, hin, hin,
                              prev_wide, wide, 1, 1, s, 0), 1))
        # remaining blocks (and the stride-1 3x3 / expand convolutions of every block)
        out.append((ConvLayer(tag + "1x1_%dto%d_at%d" % (wide, mid, hw), batch, hw, hw, wide, mid, 1, 1, 1, 0), blocks - 1))
        out.append((ConvLayer(tag + "3x3_%dto%d_at%d" % (mid, mid, hw), batch, hw, hw, mid, mid, 3, 3, 1, 1),
                    blocks if s == 1 else blocks - 1))
        out.append((ConvLayer(tag + "1x1_%dto%d_at%d" % (mid, wide, hw), batch, hw, hw, mid, wide, 1, 1, 1, 0), blocks))
        prev_wide = wide
    return out


def resnet18_layers(batch: int = 256) -> List[ConvLayer]:
    """Distinct convolutions of the ResNet-18 basic-block stages (Section 4 trains it on ImageNet): 3x3 at
    64@56, 128@28, 256@14, 512@7, the stride-2 3x3 that opens stages 2-4 and their 1x1 stride-2 shortcuts."""
    out = []
    prev = 64
    for stage, (hw, ch) in enumerate([(56, 64), (28, 128), (14, 256), (7, 512)], start=1):
        tag = "r18_s%d_" % stage
        if stage > 1:
            out.append(ConvLayer(tag + "3x3s2_%dto%d_at%d" % (prev, ch, 2 * hw), batch, 2 * hw, 2 * hw, prev, ch, 3, 3, 2, 1))
            out.append(ConvLayer(tag + "projs2_%dto%d_at%d" % (prev, ch, 2 * hw), batch, 2 * hw, 2 * hw, prev, ch, 1, 1, 2, 0))
        out.append(ConvLayer(tag + "3x3_%dto%d_at%d" % (ch, ch, hw), batch, hw, hw, ch, ch, 3, 3, 1, 1))
        prev = ch
    return out


def regnetx_400mf_layer_counts(batch: int = 256):
    """Distinct convolutions of the RegNetX-400MF body (Section 4 trains it on ImageNet) with the number of times
    the network holds each: stage widths 32, 64, 160, 384 at 56, 28, 14, 7 pixels, depths 1, 2, 7, 12, group width
    16 (so 2, 4, 10, 24 groups), bottleneck ratio 1. A block is 1x1 -> grouped 3x3 -> 1x1; the first block of a
    stage takes the previous stage's width at twice the resolution, strides in its 3x3 and has a 1x1 stride-2
    shortcut."""
    out = []
    prev = 32
    for stage, (hw, ch, depth) in enumerate([(56, 32, 1), (28, 64, 2), (14, 160, 7), (7, 384, 12)], start=1):
        tag = "rx_s%d_" % stage
        g = ch // 16
        out.append((ConvLayer(tag + "1x1_%dto%d_at%d" % (prev, ch, 2 * hw), batch, 2 * hw, 2 * hw, prev, ch, 1, 1, 1, 0), 1))
        out.append((ConvLayer(tag + "3x3s2g%d_%d_at%d" % (g, ch, 2 * hw), batch, 2 * hw, 2 * hw, ch, ch, 3, 3, 2, 1, g), 1))
        out.append((ConvLayer(tag + "projs2_%dto%d_at%d" % (prev, ch, 2 * hw), batch, 2 * hw, 2 * hw, prev, ch, 1, 1, 2, 0), 1))
        out.append((ConvLayer(tag + "1x1_%dto%d_at%d" % (ch, ch, hw), batch, hw, hw, ch, ch, 1, 1, 1, 0), 2 * depth - 1))
        if depth > 1:
            out.append((ConvLayer(tag + "3x3g%d_%d_at%d" % (g, ch, hw), batch, hw, hw, ch, ch, 3, 3, 1, 1, g), depth - 1))
        prev = ch
    return out


def regnetx_400mf_layers(batch: int = 256) -> List[ConvLayer]:
    return [layer for layer, _ in regnetx_400mf_layer_counts(batch)]


def conv_layer_tensors(layer: ConvLayer, seed: int):
    """(dO, W) for one layer: dO = ReLU-masked Laplace, W = He-normal N(0, 2/(R*S*Cin))."""
    dO = relu_masked_laplace_bf16(layer.dO_shape(), seed, stream=1)
    W = normal_bf16(layer.W_shape(), float(np.sqrt(2.0 / (layer.R * layer.S * (layer.Cin // layer.groups)))), seed, stream=2)
    return dO, W


def fc_tensors(rows: int, K: int, N: int, seed: int):
    """(dO, W) for a fully connected layer: dO ~ N(0,1), W ~ N(0, 1/K)."""
    dO = normal_bf16((rows, K), 1.0, seed, stream=1)
    W = normal_bf16((K, N), float(1.0 / np.sqrt(K)), seed, stream=2)
    return dO, W


FC_SMALL = dict(rows=256, K=512, N=256, seed=0)
GEMM_LARGE = dict(rows=16384, K=4096, N=4096, seed=0)
NM_SWEEP = [(1, 4), (2, 4), (2, 8), (2, 16)]
