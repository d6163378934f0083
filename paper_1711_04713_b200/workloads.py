"""Seeded synthetic inputs and layer shapes of the workloads.

Holds no arithmetic of the method: only shapes and random fp32 tensors.  Every
tensor is drawn on the host from a seeded ``torch.Generator`` so that the CPU
oracle and the CUDA path are handed identical arrays.

The shapes stand in for the networks the paper studies (VGG16 on ImageNet,
Sec. 2.2-2.5); the dataset and trained weights are not needed for the forward
pass of the low-precision layers and are replaced by He-normal weights and
normal / uniform inputs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

# VGG16 convolution stack: (name, H=W of the input, Cin, Cout); 3x3, pad 1, stride 1.
VGG16_CONV = [
    ("conv1_1", 224, 3, 64), ("conv1_2", 224, 64, 64),
    ("conv2_1", 112, 64, 128), ("conv2_2", 112, 128, 128),
    ("conv3_1", 56, 128, 256), ("conv3_2", 56, 256, 256), ("conv3_3", 56, 256, 256),
    ("conv4_1", 28, 256, 512), ("conv4_2", 28, 512, 512), ("conv4_3", 28, 512, 512),
    ("conv5_1", 14, 512, 512), ("conv5_2", 14, 512, 512), ("conv5_3", 14, 512, 512),
]
VGG16_POOL_AFTER = {"conv1_2", "conv2_2", "conv3_3", "conv4_3", "conv5_3"}
VGG16_FC = [("fc6", 25088, 4096, True), ("fc7", 4096, 4096, True), ("fc8", 4096, 1000, False)]


def vgg16_macs_per_image() -> int:
    macs = sum(h * h * cout * 9 * cin for _, h, cin, cout in VGG16_CONV)
    macs += sum(k * o for _, k, o, _ in VGG16_FC)
    return macs


@dataclass
class LayerSpec:
    type: str                 # "conv" | "ip" | "pool"
    name: str = ""
    cin: int = 0
    cout: int = 0
    ksize: int = 0
    pad: int = 0
    stride: int = 1
    relu: bool = True
    extra: dict = field(default_factory=dict)


def vgg16_specs() -> list[LayerSpec]:
    specs: list[LayerSpec] = []
    for name, _, cin, cout in VGG16_CONV:
        specs.append(LayerSpec("conv", name, cin, cout, 3, 1, 1, True))
        if name in VGG16_POOL_AFTER:
            specs.append(LayerSpec("pool", "pool" + name[4]))
    for name, k, o, relu in VGG16_FC:
        specs.append(LayerSpec("ip", name, k, o, relu=relu))
    return specs


# Giga1Net (paper, "New Benchmark Networks", Table 1): (Cin, Cout, kernel, input H=W, pool after, pad).
# The table lists no paddings; these are the ones that reproduce its input sizes (112 -> 7x7 ->
# pool gives the listed 54 only with pad 1; the 18x18 maps are kept through the 3x3 layers by pad 1)
# and its cost of about 1 GOp per frame (567 MMAC with the first inner product fed by 9 x 9 x 128).
GIGA1NET_CONV = [
    (3, 16, 1, 224, True, 0), (16, 16, 7, 112, True, 1), (16, 32, 7, 54, True, 0),
    (32, 64, 5, 24, False, 1), (64, 64, 5, 22, False, 1), (64, 64, 5, 20, False, 1),
    (64, 128, 3, 18, False, 1), (128, 128, 3, 18, False, 1), (128, 128, 3, 18, False, 1),
    (128, 128, 3, 18, False, 1), (128, 128, 3, 18, True, 1),
]
GIGA1NET_FC = [("fc12", 9 * 9 * 128, 4096, True), ("fc13", 4096, 1000, False)]


def giga1net_specs() -> list[LayerSpec]:
    specs: list[LayerSpec] = []
    for i, (cin, cout, k, _, pool, pad) in enumerate(GIGA1NET_CONV, start=1):
        specs.append(LayerSpec("conv", f"conv{i}", cin, cout, k, pad, 1, True))
        if pool:
            specs.append(LayerSpec("pool", f"pool{i}"))
    for name, k, o, relu in GIGA1NET_FC:
        specs.append(LayerSpec("ip", name, k, o, relu=relu))
    return specs


def giga1net_macs_per_image() -> int:
    macs = 0
    for cin, cout, k, h, _, pad in GIGA1NET_CONV:
        oh = h + 2 * pad - k + 1
        macs += oh * oh * cout * k * k * cin
    return macs + sum(k * o for _, k, o, _ in GIGA1NET_FC)


def lenet_specs() -> list[LayerSpec]:
    return [
        LayerSpec("conv", "conv1", 1, 20, 5, 0, 1, True), LayerSpec("pool", "pool1"),
        LayerSpec("conv", "conv2", 20, 50, 5, 0, 1, True), LayerSpec("pool", "pool2"),
        LayerSpec("ip", "ip1", 800, 500, relu=True), LayerSpec("ip", "ip2", 500, 10, relu=False),
    ]


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def normal(shape, std: float, seed: int) -> np.ndarray:
    return (torch.randn(shape, generator=_gen(seed), dtype=torch.float32) * std).numpy()


def uniform01(shape, seed: int) -> np.ndarray:
    return torch.rand(shape, generator=_gen(seed), dtype=torch.float32).numpy()


def relu_normal(shape, seed: int) -> np.ndarray:
    """max(N(0,1), 0): about half zeros, like post-ReLU activations."""
    return torch.randn(shape, generator=_gen(seed), dtype=torch.float32).clamp_(min=0).numpy()


def he_conv_weight(cout: int, r: int, s: int, cin: int, seed: int) -> np.ndarray:
    """[Cout][R][S][Cin], N(0, 2/fan_in)."""
    return normal((cout, r, s, cin), math.sqrt(2.0 / (r * s * cin)), seed)


def he_ip_weight(o: int, k: int, seed: int) -> np.ndarray:
    return normal((o, k), math.sqrt(2.0 / k), seed)


def bias(n: int, seed: int) -> np.ndarray:
    """N(0, sigma = 0.01)."""
    return normal((n,), 0.01, seed)


def make_params(specs: list[LayerSpec], seed: int) -> list[dict]:
    """fp32 parameters for a stack; one independent stream per layer."""
    out = []
    for i, sp in enumerate(specs):
        if sp.type == "conv":
            out.append({"type": "conv", "name": sp.name,
                        "w": he_conv_weight(sp.cout, sp.ksize, sp.ksize, sp.cin, seed * 1000 + 2 * i + 1),
                        "b": bias(sp.cout, seed * 1000 + 2 * i + 2),
                        "pad": sp.pad, "stride": sp.stride, "relu": sp.relu})
        elif sp.type == "ip":
            out.append({"type": "ip", "name": sp.name,
                        "w": he_ip_weight(sp.cout, sp.cin, seed * 1000 + 2 * i + 1),
                        "b": bias(sp.cout, seed * 1000 + 2 * i + 2), "relu": sp.relu})
        else:
            out.append({"type": "pool", "name": sp.name})
    return out


def lenet_input(batch: int, seed: int) -> np.ndarray:
    """NHWC batch x 28 x 28 x 1, uniform [0, 1)."""
    return uniform01((batch, 28, 28, 1), seed)


def vgg16_input(batch: int, seed: int, hw: int = 224) -> np.ndarray:
    """NHWC batch x hw x hw x 3, N(0, 1) per channel."""
    return normal((batch, hw, hw, 3), 1.0, seed)
