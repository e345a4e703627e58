"""Convolution-layer lists of the Fixup ResNets the EOQ paper trains (arXiv 2105.13890, Sec. 5.1), as synthetic workloads.

A workload is the ordered list of quantized convolution layers of one network at one batch size.  Each entry
carries the geometry the C ABI needs plus what the Fixup layer unit around the convolution does (Sec. 3.1 and
3.2.1): whether a ReLU follows, whether a shortcut joins before it, whether gamma is trainable (then x2 is
kept for g_gamma), whether the layer sits in a residual branch (then its Kaiming weights are scaled by
L^(-1/(2m-2))), and whether an error has to be propagated to its input (not for the first layer).
Channel counts are padded to multiples of 16 for the kernels (8 for the RGB input of a 7x7 first layer);
`c_in_true` keeps the real count for op counting.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


@dataclass(frozen=True)
class Layer:
    name: str
    n: int
    h: int
    w: int
    c_in: int
    c_out: int
    k: int
    stride: int
    pad: int
    c_in_true: int
    relu: bool = True
    shortcut: bool = False
    gamma_trainable: bool = False
    in_branch: bool = True
    has_dgrad: bool = True

    @property
    def ho(self) -> int:
        return (self.h + 2 * self.pad - self.k) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 * self.pad - self.k) // self.stride + 1

    @property
    def macs(self) -> int:
        """Multiply-accumulates of one pass (forward, dgrad and wgrad all do this many)."""
        return self.n * self.ho * self.wo * self.c_out * self.c_in_true * self.k * self.k

    @property
    def passes(self) -> int:
        return 3 if self.has_dgrad else 2

    @property
    def weight_elems(self) -> int:
        return self.c_out * self.k * self.k * self.c_in


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    layers: List[Layer]
    L: int  # residual blocks
    m: int  # layers per block

    @property
    def total_macs(self) -> int:
        return sum(l.macs * l.passes for l in self.layers)

    @property
    def total_ops(self) -> int:
        return 2 * self.total_macs


def fixup_alpha(L: int, m: int) -> float:
    """Layer-wise coefficient of Fixup initialisation, L^(-1/(2m-2)) (Sec. 3.1, Eq. 1)."""
    return float(L) ** (-1.0 / (2 * m - 2))


def init_weight_f32(layer: Layer, wl: Workload, normal_draws: np.ndarray) -> np.ndarray:
    """fp32 weights [c_out,k,k,c_in] from N(0,1) draws: Kaiming std sqrt(2/n) (Sec. 4), alpha in branches (Sec. 3.2.3).
    Padding input channels get zero weights."""
    fan_in = layer.c_in_true * layer.k * layer.k
    std = np.sqrt(2.0 / fan_in) * (fixup_alpha(wl.L, wl.m) if layer.in_branch else 1.0)
    w = (np.asarray(normal_draws, dtype=np.float64) * std).astype(np.float32)
    if layer.c_in_true < layer.c_in:
        w[..., layer.c_in_true:] = 0.0
    return w


def _pad16(c: int) -> int:
    return (c + 15) // 16 * 16


def _basic_stage(layers, name, n, h, c_in, c_out, blocks, stride):
    """A stage of basic blocks: unit A (conv, gamma fixed, ReLU) then unit B (conv, gamma, shortcut, ReLU)."""
    for b in range(blocks):
        s = stride if b == 0 else 1
        ci = c_in if b == 0 else c_out
        layers.append(Layer(f"{name}.{b}.a", n, h, h, ci, c_out, 3, s, 1, ci))
        if s != 1 or ci != c_out:
            layers.append(Layer(f"{name}.{b}.proj", n, h, h, ci, c_out, 1, s, 0, ci, relu=False, in_branch=False))
        h = (h + 2 - 3) // s + 1
        layers.append(Layer(f"{name}.{b}.b", n, h, h, c_out, c_out, 3, 1, 1, c_out, shortcut=True, gamma_trainable=True))
    return h


# The RGB input of a 7x7 stride-2 first layer is stored with 8 channels (3 real): the library's filter-row path
# takes 8- or 16-channel inputs and a filter row of 8 pixels is then a 64-byte K slice instead of 128.
STEM_CHANNELS = 8


def _imagenet_basic(name: str, blocks, batch: int, image: int) -> Workload:
    """ImageNet-shaped ResNet of basic blocks: 7x7 stride-2 first layer, 3x3 stride-2 max-pool, four stages."""
    layers: List[Layer] = []
    layers.append(Layer("stem", batch, image, image, STEM_CHANNELS, 64, 7, 2, 3, 3, in_branch=False, has_dgrad=False))
    h = (image + 6 - 7) // 2 + 1
    h = (h + 2 - 3) // 2 + 1  # 3x3 stride-2 max-pool
    c = 64
    for i, (co, s) in enumerate(((64, 1), (128, 2), (256, 2), (512, 2))):
        h = _basic_stage(layers, f"layer{i + 1}", batch, h, c, co, blocks[i], s)
        c = co
    return Workload(f"fixup_{name}_b{batch}_{image}", batch, layers, L=sum(blocks), m=2)


def resnet18(batch: int = 64, image: int = 224) -> Workload:
    return _imagenet_basic("resnet18", (2, 2, 2, 2), batch, image)


def resnet34(batch: int = 64, image: int = 224) -> Workload:
    """ResNet-34, the second ImageNet network of Sec. 5.1: basic blocks [3, 4, 6, 3], L = 16."""
    return _imagenet_basic("resnet34", (3, 4, 6, 3), batch, image)


def resnet20(batch: int = 128, image: int = 32) -> Workload:
    layers: List[Layer] = []
    layers.append(Layer("stem", batch, image, image, _pad16(3), 16, 3, 1, 1, 3, in_branch=False, has_dgrad=False))
    h, c = image, 16
    for i, (co, s) in enumerate(((16, 1), (32, 2), (64, 2))):
        h = _basic_stage(layers, f"stage{i + 1}", batch, h, c, co, 3, s)
        c = co
    return Workload(f"fixup_resnet20_b{batch}_{image}", batch, layers, L=9, m=2)


def resnet110(batch: int = 128, image: int = 32) -> Workload:
    """ResNet-110 on CIFAR-shaped input, the network of the small-batch experiment (Sec. 5.4): three stages of
    18 basic blocks with 16 / 32 / 64 channels, L = 54."""
    layers: List[Layer] = []
    layers.append(Layer("stem", batch, image, image, _pad16(3), 16, 3, 1, 1, 3, in_branch=False, has_dgrad=False))
    h, c = image, 16
    for i, (co, s) in enumerate(((16, 1), (32, 2), (64, 2))):
        h = _basic_stage(layers, f"stage{i + 1}", batch, h, c, co, 18, s)
        c = co
    return Workload(f"fixup_resnet110_b{batch}_{image}", batch, layers, L=54, m=2)


def resnet50(batch: int = 32, image: int = 224) -> Workload:
    layers: List[Layer] = []
    layers.append(Layer("stem", batch, image, image, STEM_CHANNELS, 64, 7, 2, 3, 3, in_branch=False, has_dgrad=False))
    h = (image + 6 - 7) // 2 + 1
    h = (h + 2 - 3) // 2 + 1
    c = 64
    for i, (mid, blocks, s) in enumerate(((64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2))):
        out = mid * 4
        for b in range(blocks):
            st = s if b == 0 else 1
            ci = c if b == 0 else out
            layers.append(Layer(f"layer{i + 1}.{b}.a", batch, h, h, ci, mid, 1, 1, 0, ci))
            layers.append(Layer(f"layer{i + 1}.{b}.b", batch, h, h, mid, mid, 3, st, 1, mid))
            if b == 0:
                layers.append(Layer(f"layer{i + 1}.{b}.proj", batch, h, h, ci, out, 1, st, 0, ci, relu=False, in_branch=False))
            h2 = (h + 2 - 3) // st + 1
            layers.append(Layer(f"layer{i + 1}.{b}.c", batch, h2, h2, mid, out, 1, 1, 0, mid, shortcut=True, gamma_trainable=True))
            h = h2
        c = out
    return Workload(f"fixup_resnet50_b{batch}_{image}", batch, layers, L=16, m=3)


def single_layer() -> Workload:
    """The single 3x3 layer: N=8, 16 -> 16 channels, 32x32."""
    return Workload("single_conv3x3_n8_c16_32x32", 8, [Layer("conv", 8, 32, 32, 16, 16, 3, 1, 1, 16, in_branch=False)], L=1, m=2)


def layer64(batch: int = 512) -> Workload:
    """Two 3x3 stride-1 layers of the ResNet-18 first stage (64 -> 64 channels, 56x56): the profiling case.

    At batch 512 each activation tensor is 103 MB, so a layer's tensors do not fit in a B200's L2.  The first
    layer takes the quantized image (device-side input exponent), the second is an ordinary inner layer.
    """
    layers = [Layer("conv.a", batch, 56, 56, 64, 64, 3, 1, 1, 64, in_branch=False, has_dgrad=False),
              Layer("conv.b", batch, 56, 56, 64, 64, 3, 1, 1, 64, in_branch=False)]
    return Workload(f"conv3x3_c64_56x56_b{batch}_x2", batch, layers, L=1, m=2)


def get(name: str, batch: int | None = None) -> Workload:
    table = {"single": single_layer, "layer64": layer64, "resnet20": resnet20, "resnet18": resnet18, "resnet34": resnet34,
             "resnet50": resnet50, "resnet110": resnet110}
    fn = table[name]
    if name == "single" or batch is None:
        return fn()
    return fn(batch)
