"""Seeded synthetic workloads shaped like the paper's networks.

This module only *describes* layers and draws random tensors.  It holds none of the
method's arithmetic (no pattern library, no projection, no packing, no convolution), so
both the CUDA path and the CPU oracle may be fed from it without sharing any logic.

Shapes follow the paper's evaluated networks (VGG-16 and ResNet-50 on 224x224 ImageNet
images, Section 7); weights and images are synthetic stand-ins:

* weights  ~ N(0, sigma^2), sigma = sqrt(2 / (9 * C_in)), layout [F][C][3][3], fp32
* inputs   = max(0, N(0,1)), layout NHWC, fp32 (optionally rounded to fp16 by the caller)

Generator: numpy ``Generator(PCG64(seed))``; weights are drawn first, then inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from fractions import Fraction
from typing import List, Optional

import numpy as np

BASE_SEED = 20200107


@dataclass(frozen=True)
class Layer:
    """One 3x3 convolution layer: input H x W x C, output F filters, stride 1 or 2, pad 1."""
    name: str
    H: int
    W: int
    C: int
    F: int
    stride: int = 1
    dense: bool = False          # True: not pruned (all 9 taps of all F*C kernels)
    keep: Fraction = Fraction(1)  # fraction of kernels kept by connectivity pruning
    K: int = 8                   # pattern-library size
    index: int = 0               # position in its config (used for seeding)
    cell: int = 0                # sweep-cell number (config 4)

    @property
    def Ho(self) -> int:
        return (self.H + 2 - 3) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 - 3) // self.stride + 1

    @property
    def n_keep(self) -> int:
        """Number of kernels kept: floor(F*C*keep) in exact integer arithmetic."""
        if self.dense:
            return self.F * self.C
        return (self.F * self.C * self.keep.numerator) // self.keep.denominator

    def taps(self) -> int:
        return 9 if self.dense else 4

    def useful_flop(self, N: int) -> int:
        """2 * useful multiply-accumulates (only stored taps count)."""
        return 2 * N * self.Ho * self.Wo * self.taps() * self.n_keep

    def dense_flop(self, N: int) -> int:
        return 2 * N * self.Ho * self.Wo * 9 * self.F * self.C

    def compulsory_bytes(self, N: int, elem: int) -> int:
        """Input once + output once + stored taps and channel indices once."""
        blob = self.n_keep * (self.taps() * elem + 2)
        return N * self.H * self.W * self.C * elem + N * self.Ho * self.Wo * self.F * elem + blob


@dataclass(frozen=True)
class Config:
    number: int
    name: str
    N: int
    dtype: str                    # "f32" | "f16" (storage type; accumulation is fp32)
    layers: List[Layer] = field(default_factory=list)


_VGG_CH = [64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]
_VGG_HW = [224, 224, 112, 112, 56, 56, 56, 28, 28, 28, 14, 14, 14]


def _vgg_layers(keep: Fraction) -> List[Layer]:
    out = []
    cin = 3
    for i, (f, hw) in enumerate(zip(_VGG_CH, _VGG_HW)):
        out.append(Layer(name=f"conv{i + 1}", H=hw, W=hw, C=cin, F=f, stride=1,
                         dense=(i == 0), keep=keep, K=8, index=i))
        cin = f
    return out


def _resnet50_layers(keep: Fraction) -> List[Layer]:
    out = []
    idx = 0
    prev_hw = 56
    for ch, hw, reps in [(64, 56, 3), (128, 28, 4), (256, 14, 6), (512, 7, 3)]:
        for r in range(reps):
            first_of_later_stage = (r == 0 and ch != 64)
            stride = 2 if first_of_later_stage else 1
            hin = prev_hw if first_of_later_stage else hw
            out.append(Layer(name=f"res{ch}_{r}", H=hin, W=hin, C=ch, F=ch, stride=stride,
                             keep=keep, K=8, index=idx))
            idx += 1
        prev_hw = hw
    return out


def _sweep_layers() -> List[Layer]:
    out = []
    cell = 0
    for K in (4, 8, 12):
        for keep in (Fraction(1), Fraction(1, 2), Fraction(1, 8)):
            out.append(Layer(name=f"sweep_K{K}_keep{keep.numerator}of{keep.denominator}",
                             H=28, W=28, C=256, F=256, keep=keep, K=K, index=0, cell=cell))
            cell += 1
    return out


def configs() -> List[Config]:
    """The five evaluation configurations."""
    return [
        Config(0, "single 56x56x64->64 fp32 batch 1, keep 30%", 1, "f32",
               [Layer("single", 56, 56, 64, 64, keep=Fraction(3, 10), K=8, index=0)]),
        Config(1, "VGG-16 conv stack fp32 batch 1, keep 12.5%", 1, "f32", _vgg_layers(Fraction(1, 8))),
        Config(2, "ResNet-50 3x3 layers fp32 batch 32, keep 25%", 32, "f32", _resnet50_layers(Fraction(1, 4))),
        Config(3, "VGG-16 conv stack fp16 storage batch 64, keep 12.5%", 64, "f16", _vgg_layers(Fraction(1, 8))),
        Config(4, "sweep 28x28x256->256 fp32 batch 32", 32, "f32", _sweep_layers()),
    ]


def layer_seed(config: int, layer: Layer) -> int:
    return BASE_SEED * 10000 + config * 1000 + layer.cell * 100 + layer.index


def make_weights(rng: np.random.Generator, F: int, C: int) -> np.ndarray:
    sigma = np.sqrt(2.0 / (9.0 * C))
    return (rng.standard_normal((F, C, 3, 3)) * sigma).astype(np.float32)


def make_inputs(rng: np.random.Generator, N: int, H: int, W: int, C: int) -> np.ndarray:
    x = rng.standard_normal((N, H, W, C), dtype=np.float32)
    np.maximum(x, 0.0, out=x)
    return x


def make_layer_tensors(config: int, layer: Layer, N: int, n_limit: Optional[int] = None):
    """(weights [F][C][3][3] fp32, inputs [N'][H][W][C] fp32), N' = min(N, n_limit)."""
    rng = np.random.Generator(np.random.PCG64(layer_seed(config, layer)))
    w = make_weights(rng, layer.F, layer.C)
    n = N if n_limit is None else min(N, n_limit)
    x = make_inputs(rng, n, layer.H, layer.W, layer.C)
    return w, x
