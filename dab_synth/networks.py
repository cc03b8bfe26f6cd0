"""Layer lists of the three network shapes the paper trains (Section 5.1), with seeded random weights.

Shapes and numbers only: no arithmetic of the method.  A layer is a dict with "kind" in
  conv_dense   full-precision convolution (first layer, last classifier, 1x1 shortcut projections): w [Cout x C*kh*kw],
               optional bias; kh, kw, stride, pad
  conv_binary  a binarized layer: w [Cout x C*kh*kw] full precision, coded per filter by whoever runs the chain
  affine       per-channel scale and shift (a folded normalisation layer)
  relu, maxpool (kh, kw, stride, pad), save (remember the running tensor for a shortcut), add (running + remembered)
and "on_saved": True where a layer transforms the remembered tensor instead of the running one.
Fully connected layers are convolutions whose kernel covers their whole input.  The networks are the paper's
only in shape: Sketch-A-Net (all but first and last layer binarized), an AlexNet-like net, and a ResNet-18-like
net whose 16 3x3 convolutions are binarized (global max pooling stands in for its average pooling).
"""
from __future__ import annotations

import numpy as np

from . import DEFAULT_SEED, normal, stroke_batch, uniform01


class _Builder:
    def __init__(self, seed: int, c: int):
        self.seed, self.c, self.k, self.layers = seed, c, 0, []

    def _stream(self) -> int:
        self.k += 1
        return 7000 + self.k

    def conv(self, kind, cout, kh, kw, stride=1, pad=0, bias=False, on_saved=False, c_in=None):
        c = self.c if c_in is None else c_in
        n = c * kh * kw
        std = float(np.sqrt(2.0 / n))
        layer = {"kind": kind, "w": normal((cout, n), std, self.seed, self._stream()), "kh": kh, "kw": kw,
                 "stride": (stride, stride), "pad": (pad, pad), "Cout": cout}
        if bias:
            layer["bias"] = normal((cout,), 0.1, self.seed, self._stream())
        if on_saved:
            layer["on_saved"] = True
        else:
            self.c = cout
        self.layers.append(layer)
        return self

    def affine(self, on_saved=False, channels=None):
        c = self.c if channels is None else channels
        scale = (0.5 + uniform01(self.seed, self._stream(), 0, c)).astype(np.float32)
        shift = normal((c,), 0.1, self.seed, self._stream())
        layer = {"kind": "affine", "scale": scale, "shift": shift}
        if on_saved:
            layer["on_saved"] = True
        self.layers.append(layer)
        return self

    def relu(self):
        self.layers.append({"kind": "relu"})
        return self

    def maxpool(self, k, stride, pad=0):
        self.layers.append({"kind": "maxpool", "kh": k, "kw": k, "stride": (stride, stride), "pad": (pad, pad)})
        return self

    def save(self):
        self.layers.append({"kind": "save"})
        return self

    def add(self):
        self.layers.append({"kind": "add"})
        return self


def sketch_a_net(seed: int = DEFAULT_SEED):
    """Input 1 x 225 x 225.  conv1 15x15 s3 (full precision), binarized conv2 5x5, conv3/4/5 3x3, fc6 7x7, fc7, fc8 full."""
    b = _Builder(seed, 1)
    b.conv("conv_dense", 64, 15, 15, 3).relu().maxpool(3, 2)                 # 225 -> 71 -> 35
    b.conv("conv_binary", 128, 5, 5).relu().maxpool(3, 2)                    # 35 -> 31 -> 15
    b.conv("conv_binary", 256, 3, 3, 1, 1).relu()
    b.conv("conv_binary", 256, 3, 3, 1, 1).relu()
    b.conv("conv_binary", 256, 3, 3, 1, 1).relu().maxpool(3, 2)              # 15 -> 7
    b.conv("conv_binary", 512, 7, 7).relu()                                  # fc6
    b.conv("conv_binary", 512, 1, 1).relu()                                  # fc7
    b.conv("conv_dense", 250, 1, 1, bias=True)                               # fc8
    return b.layers, (1, 225, 225)


def alexnet_like(seed: int = DEFAULT_SEED):
    """Input 3 x 224 x 224.  conv1 11x11 s4 (full precision), binarized conv2..5 and two 4096-wide layers, classifier full."""
    b = _Builder(seed + 1, 3)
    b.conv("conv_dense", 96, 11, 11, 4, 2).relu().maxpool(3, 2)              # 224 -> 55 -> 27
    b.affine().conv("conv_binary", 256, 5, 5, 1, 2).relu().maxpool(3, 2)     # 27 -> 13
    b.affine().conv("conv_binary", 384, 3, 3, 1, 1).relu()
    b.affine().conv("conv_binary", 384, 3, 3, 1, 1).relu()
    b.affine().conv("conv_binary", 256, 3, 3, 1, 1).relu().maxpool(3, 2)     # 13 -> 6
    b.affine().conv("conv_binary", 4096, 6, 6).relu()
    b.affine().conv("conv_binary", 4096, 1, 1).relu()
    b.conv("conv_dense", 250, 1, 1, bias=True)
    return b.layers, (3, 224, 224)


def resnet18_like(seed: int = DEFAULT_SEED):
    """Input 3 x 224 x 224.  Full-precision 7x7 stem, 8 residual blocks of two binarized 3x3 convolutions (64, 128,
    256, 512 channels; 1x1 full-precision projections where the shape changes), global max pooling, classifier."""
    b = _Builder(seed + 2, 3)
    b.conv("conv_dense", 64, 7, 7, 2, 3).affine().relu().maxpool(3, 2, 1)    # 224 -> 112 -> 56
    for stage, c in enumerate((64, 128, 256, 512)):
        for block in range(2):
            stride = 2 if (stage > 0 and block == 0) else 1
            c_in = b.c
            b.save()
            b.affine().conv("conv_binary", c, 3, 3, stride, 1).relu()
            b.affine().conv("conv_binary", c, 3, 3, 1, 1)
            if stride != 1 or c_in != c:
                b.conv("conv_dense", c, 1, 1, stride, 0, on_saved=True, c_in=c_in).affine(on_saved=True, channels=c)
            b.add().relu()
    b.maxpool(7, 1)
    b.conv("conv_dense", 250, 1, 1, bias=True)
    return b.layers, (3, 224, 224)


def network_input(shape, batch: int, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """Sparse stroke images (background 0, about 5 % of the pixels 1), replicated over the input channels."""
    c, h, w = shape
    return stroke_batch(batch, c, h, w, seed, 9000 + stream)


def googlenet_branch_layers(batch: int = 8):
    """Binarized layer shapes of GoogLeNet-style inception branches (1x1, 3x3 and 5x5 kernels on one input), as
    (name, N, C, H, W, Cout, kh, kw, stride, pad) tuples: a second set of layer shapes beside the five configs."""
    return [("3a_1x1", batch, 192, 28, 28, 64, 1, 1, 1, 0), ("3a_3x3", batch, 96, 28, 28, 128, 3, 3, 1, 1),
            ("3a_5x5", batch, 16, 28, 28, 32, 5, 5, 1, 2), ("4a_3x3", batch, 96, 14, 14, 208, 3, 3, 1, 1),
            ("4a_5x5", batch, 16, 14, 14, 48, 5, 5, 1, 2), ("5a_3x3", batch, 160, 7, 7, 320, 3, 3, 1, 1),
            ("5a_5x5", batch, 32, 7, 7, 128, 5, 5, 1, 2)]
