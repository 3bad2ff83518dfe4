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


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}
