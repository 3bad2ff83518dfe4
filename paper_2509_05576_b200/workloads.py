"""Seeded synthetic layers shaped like the paper's workloads.

This module only draws random inputs (numpy ``PCG64``); it contains none of the method's
arithmetic, so both the CUDA tests and the CPU oracle's tests may use it.  The synthetic
layers stand in for the ImageNet / COCO calibration activations and the trained ResNet /
YOLOv5 weights the paper measures on (Sec. 6), which are not available offline: only layer
shapes and coarse activation statistics (non-negative post-ReLU, SiLU-shaped, sparse) are kept.

Recipe: ``rng = Generator(PCG64(seed))``; W is drawn first, then X; both float32.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class LayerSpec:
    name: str
    rows: int          # d_row = Cout
    cols: int          # d_col = Cin * k * k
    n: int             # calibration columns
    bits: int
    w_dist: str        # "normal0.02" | "kaiming"
    x_dist: str        # "halfnormal" | "halfnormal_sparse30" | "silu" | "normal"
    seed: int
    damp: float = 0.01  # relative: lambda = damp * mean(diag H)

    @property
    def weights(self) -> int:
        return self.rows * self.cols


def make_layer(spec: LayerSpec):
    """Returns (W [rows, cols] float32, X [cols, n] float32)."""
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    if spec.w_dist == "normal0.02":
        W = rng.standard_normal((spec.rows, spec.cols)) * 0.02
    elif spec.w_dist == "kaiming":
        W = rng.standard_normal((spec.rows, spec.cols)) * np.sqrt(2.0 / spec.cols)
    else:
        raise ValueError(spec.w_dist)
    W = W.astype(np.float32)
    Z = rng.standard_normal((spec.cols, spec.n), dtype=np.float32)
    if spec.x_dist == "halfnormal":
        X = np.abs(Z)
    elif spec.x_dist == "halfnormal_sparse30":
        X = np.abs(Z)
        X[rng.random((spec.cols, spec.n), dtype=np.float32) < 0.3] = 0.0
    elif spec.x_dist == "silu":
        Zd = Z.astype(np.float64)
        X = (Zd / (1.0 + np.exp(-Zd))).astype(np.float32)
    elif spec.x_dist == "normal":
        X = Z
    else:
        raise ValueError(spec.x_dist)
    return np.ascontiguousarray(W), np.ascontiguousarray(X, dtype=np.float32)


@dataclass(frozen=True)
class ConvSpec:
    """A convolutional layer given by its input, for the front end that reads activations in place."""
    name: str
    out_channels: int
    channels: int
    kh: int
    kw: int
    stride: int
    pad: int
    height: int
    width: int
    batch: int
    bits: int
    x_dist: str        # "halfnormal" (post-ReLU) | "silu" | "normal"
    seed: int
    damp: float = 0.01

    @property
    def cols(self) -> int:
        return self.channels * self.kh * self.kw

    @property
    def out_hw(self):
        return ((self.height + 2 * self.pad - self.kh) // self.stride + 1,
                (self.width + 2 * self.pad - self.kw) // self.stride + 1)

    @property
    def n(self) -> int:
        oh, ow = self.out_hw
        return self.batch * oh * ow


def make_conv_layer(spec: ConvSpec):
    """Returns (W [out_channels, channels kh kw] float32, act [batch, channels, height, width] float32); W drawn first."""
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    W = (rng.standard_normal((spec.out_channels, spec.cols)) * np.sqrt(2.0 / spec.cols)).astype(np.float32)
    Z = rng.standard_normal((spec.batch, spec.channels, spec.height, spec.width), dtype=np.float32)
    if spec.x_dist == "halfnormal":
        act = np.abs(Z)
    elif spec.x_dist == "silu":
        Zd = Z.astype(np.float64)
        act = (Zd / (1.0 + np.exp(-Zd))).astype(np.float32)
    elif spec.x_dist == "normal":
        act = Z
    else:
        raise ValueError(spec.x_dist)
    return np.ascontiguousarray(W), np.ascontiguousarray(act, dtype=np.float32)


def conv_cases():
    """Convolutions shaped like those of the paper's networks (Sec. 6): ResNet stem and bottleneck pieces, a strided
    1x1 shortcut, the 6x6 stride-2 stem of YOLOv5; small images so that the CPU oracle finishes in seconds."""
    return [
        ConvSpec("conv.stem7x7s2", 64, 3, 7, 7, 2, 3, 40, 40, 4, 4, "normal", 7001),          # cols 147 (ragged)
        ConvSpec("conv.3x3s1", 64, 64, 3, 3, 1, 1, 14, 14, 8, 4, "halfnormal", 7002),         # cols 576
        ConvSpec("conv.3x3s2", 128, 32, 3, 3, 2, 1, 28, 28, 6, 4, "halfnormal", 7003),        # cols 288, strided
        ConvSpec("conv.1x1s1", 256, 64, 1, 1, 1, 0, 14, 14, 8, 8, "halfnormal", 7004),
        ConvSpec("conv.1x1s2", 128, 64, 1, 1, 2, 0, 28, 28, 8, 4, "halfnormal", 7005),        # shortcut
        ConvSpec("conv.yolo6x6s2", 32, 3, 6, 6, 2, 2, 64, 64, 4, 8, "silu", 7006),            # cols 108
        ConvSpec("conv.3x2s1p0", 16, 5, 3, 2, 1, 0, 9, 11, 3, 3, "normal", 7007),             # odd everything
    ]


# --------------------------------------------------------------------------------------
# Layer shape sets (rows x cols = Cout x Cin*k*k)
# --------------------------------------------------------------------------------------
def resnet50_shapes():
    """53 convolutions + the classifier of ResNet-50, in network order (25 502 912 weights)."""
    shapes = [("conv1", 64, 3 * 7 * 7)]
    cin = 64
    for s, blocks in enumerate((3, 4, 6, 3), start=1):
        P = 64 * 2 ** (s - 1)
        for b in range(blocks):
            pre = f"layer{s}.{b}"
            shapes.append((pre + ".conv1", P, cin))
            shapes.append((pre + ".conv2", P, 9 * P))
            shapes.append((pre + ".conv3", 4 * P, P))
            if b == 0:
                shapes.append((pre + ".downsample", 4 * P, cin))
            cin = 4 * P
    shapes.append(("fc", 1000, 2048))
    return shapes


def resnet_basic_shapes(blocks):
    """Convolutions + classifier of a basic-block ResNet (ResNet-18: blocks (2, 2, 2, 2); ResNet-34: (3, 4, 6, 3)),
    the other ResNets the paper evaluates (Sec. 6), in network order."""
    shapes = [("conv1", 64, 3 * 7 * 7)]
    cin = 64
    for s, nblk in enumerate(blocks, start=1):
        P = 64 * 2 ** (s - 1)
        for b in range(nblk):
            pre = f"layer{s}.{b}"
            shapes.append((pre + ".conv1", P, 9 * cin))
            shapes.append((pre + ".conv2", P, 9 * P))
            if b == 0 and cin != P:
                shapes.append((pre + ".downsample", P, cin))
            cin = P
    shapes.append(("fc", 1000, 512))
    return shapes


def resnet_conv_specs(batch=21, bits=4):
    """The distinct 3x3 / 1x1 / 7x7 convolutions of ResNet-50 as ConvSpecs at their ImageNet feature-map sizes, with a
    calibration batch that gives about 4096 output positions on the 14 x 14 maps (21 x 196 = 4116), for timing the
    front end that reads activations in place against the one that is handed the unfolded patches."""
    return [
        ConvSpec("r50.layer3.conv2", 256, 256, 3, 3, 1, 1, 14, 14, batch, bits, "halfnormal", 7201),      # 256 x 2304
        ConvSpec("r50.layer4.conv2", 512, 512, 3, 3, 1, 1, 7, 7, 4 * batch, bits, "halfnormal", 7202),    # 512 x 4608
        ConvSpec("r50.layer2.conv2", 128, 128, 3, 3, 1, 1, 28, 28, batch // 4 + 1, bits, "halfnormal", 7203),
        ConvSpec("r50.layer3.down", 1024, 512, 1, 1, 2, 0, 28, 28, batch, bits, "halfnormal", 7204),      # strided 1x1
        ConvSpec("r50.conv1", 64, 3, 7, 7, 2, 3, 224, 224, 2, bits, "normal", 7205),                      # n = 25088
    ]


_YOLOV5S_COUNTS = [
    (32, 108, 1), (64, 288, 1), (32, 64, 2), (32, 32, 1), (32, 288, 1), (64, 64, 4), (128, 576, 1),
    (64, 128, 2), (64, 576, 3), (128, 128, 7), (256, 1152, 1), (128, 256, 5), (128, 1152, 6),
    (256, 256, 5), (512, 2304, 1), (256, 512, 6), (512, 512, 2), (256, 2304, 3), (512, 1024, 1),
    (128, 512, 2), (64, 256, 2), (255, 128, 1), (255, 256, 1), (255, 512, 1),
]


def yolov5s_shapes():
    """A YOLOv5s-shaped conv stack (60 layers, 7 215 616 weights) plus the stress shape 512x4608."""
    shapes = []
    for rows, cols, count in _YOLOV5S_COUNTS:
        for c in range(count):
            shapes.append((f"y{rows}x{cols}.{c}", rows, cols))
    shapes.append(("y512x4608.extra", 512, 4608))
    return shapes


# --------------------------------------------------------------------------------------
# The five benchmark configurations
# --------------------------------------------------------------------------------------
def config1():
    return [LayerSpec("c1.linear", 64, 128, 1024, 4, "normal0.02", "halfnormal", seed=0)]


def config2():
    return [LayerSpec("c2.conv3x3", 256, 2304, 4096, 4, "kaiming", "halfnormal_sparse30", seed=2000)]


def config3():
    return [LayerSpec("c3." + nm, r, c, 4096, 4, "kaiming", "halfnormal", seed=3000 + i)
            for i, (nm, r, c) in enumerate(resnet50_shapes())]


def config4(bits=(8, 4)):
    out = []
    for b in bits:
        out += [LayerSpec(f"c4.w{b}." + nm, r, c, 8192, b, "kaiming", "silu", seed=4000 + i)
                for i, (nm, r, c) in enumerate(yolov5s_shapes())]
    return out


def config5(bits=(3, 4, 8), shapes=((1024, 1024), (2048, 4608), (4096, 4096), (4096, 11008))):
    out = []
    for i, (r, c) in enumerate(shapes):
        for b in bits:
            out.append(LayerSpec(f"c5.{r}x{c}.w{b}", r, c, 8192, b, "kaiming", "normal", seed=5000 + i))
    return out


def config6():
    """ResNet-18-shaped set, N = 4096, 4-bit (second ResNet of the paper's evaluation)."""
    return [LayerSpec("c6." + nm, r, c, 4096, 4, "kaiming", "halfnormal", seed=6000 + i)
            for i, (nm, r, c) in enumerate(resnet_basic_shapes((2, 2, 2, 2)))]


def config7():
    """ResNet-34-shaped set, N = 4096, 4-bit."""
    return [LayerSpec("c7." + nm, r, c, 4096, 4, "kaiming", "halfnormal", seed=7000 + i)
            for i, (nm, r, c) in enumerate(resnet_basic_shapes((3, 4, 6, 3)))]


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5, 6: config6, 7: config7}
