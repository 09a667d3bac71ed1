"""Seeded synthetic workloads: layer shapes and input/filter generators.

This module holds no arithmetic of the im2win method (no output-size formula,
no index map); it only names layer shapes and draws tensors.  Both the CUDA
path's callers and the CPU oracle's callers take their inputs from here, so
that the two sides see identical bits.

The layers are single convolution layers in the style of the paper's Table 1
(ResNet/VGG/AlexNet-like shapes) with zero padding added; the paper does not
say what data it ran on, so every tensor is drawn from a seeded torch CPU
generator: the input stream first, then the filter.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, asdict
from typing import Dict, Tuple

import torch


@dataclass(frozen=True)
class Layer:
    name: str
    N: int
    C: int
    H: int
    W: int
    Co: int
    Kh: int
    Kw: int
    stride: int
    pad: int
    seed: int
    x_dist: str        # "uniform_pm1" | "uniform01" | "normal01"
    f_dist: str        # "uniform_pm1" | "he_normal"
    precisions: Tuple[str, ...] = ("f32", "f16")

    def dims(self) -> Dict[str, int]:
        d = asdict(self)
        return {k: d[k] for k in ("N", "C", "H", "W", "Co", "Kh", "Kw", "stride", "pad")}

    def with_batch(self, n: int) -> "Layer":
        d = asdict(self)
        d["N"] = n
        d["precisions"] = tuple(d["precisions"])
        return Layer(**d)


def _sweep(k: int) -> Layer:
    return Layer(f"cfg5k{k}", 64, 256, 28, 28, 256, k, k, 1, (k - 1) // 2, 500 + k, "normal01", "he_normal")


LAYERS: Dict[str, Layer] = {l.name: l for l in [
    Layer("cfg1", 1, 3, 32, 32, 16, 3, 3, 1, 1, 0, "uniform_pm1", "uniform_pm1", ("f32",)),
    Layer("cfg2", 128, 64, 56, 56, 64, 3, 3, 1, 1, 2, "uniform01", "he_normal"),
    Layer("cfg3", 128, 3, 224, 224, 64, 7, 7, 2, 3, 3, "normal01", "he_normal"),
    Layer("cfg4a", 128, 256, 14, 14, 256, 3, 3, 1, 1, 40, "uniform01", "he_normal"),
    Layer("cfg4b", 128, 512, 7, 7, 512, 3, 3, 1, 1, 41, "uniform01", "he_normal"),
    Layer("cfg4c", 128, 256, 28, 28, 512, 3, 3, 2, 1, 42, "uniform01", "he_normal"),
    _sweep(1), _sweep(3), _sweep(5), _sweep(7), _sweep(11),
]}

# The twelve layers of the paper's Table 1 (all without padding), batch 256.
_T1 = [
    ("cv1", 3, 227, 96, 11, 4), ("cv2", 3, 231, 96, 11, 4), ("cv3", 3, 227, 64, 7, 2),
    ("cv4", 64, 224, 64, 7, 2), ("cv5", 96, 24, 256, 5, 1), ("cv6", 256, 12, 512, 3, 1),
    ("cv7", 3, 224, 64, 3, 1), ("cv8", 64, 112, 128, 3, 1), ("cv9", 64, 56, 64, 3, 1),
    ("cv10", 128, 28, 128, 3, 1), ("cv11", 256, 14, 256, 3, 1), ("cv12", 512, 7, 512, 3, 1),
]
TABLE1_LAYERS: Dict[str, Layer] = {
    n: Layer(n, 256, c, hw, hw, co, k, k, s, 0, 1000 + i, "normal01", "he_normal")
    for i, (n, c, hw, co, k, s) in enumerate(_T1)
}

# The layer the headline metric is quoted on (ResNet-style 3x3 layer).
BENCH_LAYER = "cfg2"


def make_inputs(layer: Layer) -> Tuple[torch.Tensor, torch.Tensor]:
    """Draw (x [N,C,H,W], filter [Co,C,Kh,Kw]) as float32 CPU tensors from the layer's seed."""
    g = torch.Generator(device="cpu")
    g.manual_seed(layer.seed)
    xs = (layer.N, layer.C, layer.H, layer.W)
    fs = (layer.Co, layer.C, layer.Kh, layer.Kw)
    if layer.x_dist == "uniform_pm1":
        x = torch.rand(xs, generator=g, dtype=torch.float32) * 2.0 - 1.0
    elif layer.x_dist == "uniform01":
        x = torch.rand(xs, generator=g, dtype=torch.float32)
    elif layer.x_dist == "normal01":
        x = torch.randn(xs, generator=g, dtype=torch.float32)
    else:
        raise ValueError(layer.x_dist)
    if layer.f_dist == "uniform_pm1":
        f = torch.rand(fs, generator=g, dtype=torch.float32) * 2.0 - 1.0
    elif layer.f_dist == "he_normal":
        std = math.sqrt(2.0 / (layer.C * layer.Kh * layer.Kw))
        f = torch.randn(fs, generator=g, dtype=torch.float32) * std
    else:
        raise ValueError(layer.f_dist)
    return x.contiguous(), f.contiguous()


def make_small_integer_inputs(layer: Layer) -> Tuple[torch.Tensor, torch.Tensor]:
    """Integer-valued tensors (x in {-2..2}, filter in {-1,0,1}) for order-independent exact sums."""
    g = torch.Generator(device="cpu")
    g.manual_seed(layer.seed + 7919)
    x = torch.randint(-2, 3, (layer.N, layer.C, layer.H, layer.W), generator=g).to(torch.float32)
    f = torch.randint(-1, 2, (layer.Co, layer.C, layer.Kh, layer.Kw), generator=g).to(torch.float32)
    return x.contiguous(), f.contiguous()
