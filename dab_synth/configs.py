"""Shapes and input recipes of the five synthetic workloads (no arithmetic of the method here).

Each binarized layer is fed its own synthetic input of the right shape and distribution
("teacher forced"): non-binarized glue between layers (first conv, pooling, normalisation,
last classifier) is outside the path, and chaining layers would make bit-exact comparison
meaningless because a one-ulp difference upstream legitimately flips a split downstream.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import DEFAULT_SEED, laplace, normal, relu_activations, dense_activations


@dataclass(frozen=True)
class ConvLayer:
    name: str
    N: int
    C: int
    H: int
    W: int
    Cout: int
    kh: int
    kw: int
    stride: int = 1
    pad: int = 0
    w_std: float = 0.02

    @property
    def n(self) -> int:
        return self.C * self.kh * self.kw

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def patches(self) -> int:
        return self.N * self.Ho * self.Wo

    @property
    def binary_ops(self) -> int:
        """2 * M * N * n: one binary multiply-accumulate counted as two operations."""
        return 2 * self.patches * self.Cout * self.n

    def x_shape(self):
        return (self.N, self.C, self.H, self.W)

    def weights(self, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
        """[Cout x C*kh*kw] fp32 ~ N(0, w_std^2), flattened in (c, kh, kw) order."""
        return normal((self.Cout, self.n), self.w_std, seed, 1000 + stream)

    def inputs(self, seed: int = DEFAULT_SEED, stream: int = 0, dense: bool = False) -> np.ndarray:
        """NCHW fp32 post-ReLU activations: half-normal with 60 % exact zeros (dense: N(0,1))."""
        if dense:
            return dense_activations(self.x_shape(), seed, 2000 + stream)
        return relu_activations(self.x_shape(), 0.6, seed, 2000 + stream)


def config1() -> list[ConvLayer]:
    """One 3x3 layer, 64 -> 64 channels, 32x32, stride 1, pad 1, batch 1 (n = 576, 1024 patches)."""
    return [ConvLayer("conv3x3_64", 1, 64, 32, 32, 64, 3, 3, 1, 1, 0.05)]


def config2() -> list[ConvLayer]:
    """Sketch-A-Net-shaped binarized layers, batch 1 (first conv and last classifier stay fp32, outside)."""
    return [ConvLayer("conv2", 1, 64, 35, 35, 128, 5, 5, 1, 0, 0.02),
            ConvLayer("conv3", 1, 128, 15, 15, 256, 3, 3, 1, 1, 0.02),
            ConvLayer("conv4", 1, 256, 15, 15, 256, 3, 3, 1, 1, 0.02),
            ConvLayer("conv5", 1, 256, 15, 15, 256, 3, 3, 1, 1, 0.02),
            ConvLayer("fc6", 1, 256, 7, 7, 512, 7, 7, 1, 0, 0.02),
            ConvLayer("fc7", 1, 512, 1, 1, 512, 1, 1, 1, 0, 0.02)]


CONFIG3_POINTS = [(m, k) for m in (1024, 4096, 8192) for k in (576, 2304, 4608)]


def config3_operands(m: int, k: int, seed: int = DEFAULT_SEED):
    """A[M x k], B[M x k] i.i.d. Laplace(0, 0.05) fp32 for the bare GEMM sweep (M = N)."""
    return laplace((m, k), 0.05, seed, 3000 + k), laplace((m, k), 0.05, seed, 4000 + k)


def config4(batch: int = 128) -> list[ConvLayer]:
    """AlexNet-shaped binarized layers (first conv and last classifier fp32, outside)."""
    return [ConvLayer("conv2", batch, 96, 27, 27, 256, 5, 5, 1, 2, 0.01),
            ConvLayer("conv3", batch, 256, 13, 13, 384, 3, 3, 1, 1, 0.01),
            ConvLayer("conv4", batch, 384, 13, 13, 384, 3, 3, 1, 1, 0.01),
            ConvLayer("conv5", batch, 384, 13, 13, 256, 3, 3, 1, 1, 0.01),
            ConvLayer("fc6", batch, 256, 6, 6, 4096, 6, 6, 1, 0, 0.01),
            ConvLayer("fc7", batch, 4096, 1, 1, 4096, 1, 1, 1, 0, 0.01)]


def config5(batch: int = 256) -> list[ConvLayer]:
    """ResNet-18-shaped stack of binarized 3x3 convolutions (stem, 1x1 shortcuts and classifier outside)."""
    L = []
    L += [ConvLayer("l1_%d" % i, batch, 64, 56, 56, 64, 3, 3, 1, 1) for i in range(4)]
    L += [ConvLayer("l2_0", batch, 64, 56, 56, 128, 3, 3, 2, 1)]
    L += [ConvLayer("l2_%d" % i, batch, 128, 28, 28, 128, 3, 3, 1, 1) for i in range(1, 4)]
    L += [ConvLayer("l3_0", batch, 128, 28, 28, 256, 3, 3, 2, 1)]
    L += [ConvLayer("l3_%d" % i, batch, 256, 14, 14, 256, 3, 3, 1, 1) for i in range(1, 4)]
    L += [ConvLayer("l4_0", batch, 256, 14, 14, 512, 3, 3, 2, 1)]
    L += [ConvLayer("l4_%d" % i, batch, 512, 7, 7, 512, 3, 3, 1, 1) for i in range(1, 4)]
    return L
