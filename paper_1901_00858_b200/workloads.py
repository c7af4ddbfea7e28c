"""Seeded synthetic workloads: layer shapes and input tensors.

This module serves both the CUDA path's tests/bench and the CPU oracle's tests.  It holds
no arithmetic of the convolution itself: plane sizes are written out per layer (not derived
from the output-size formula) and tensors are drawn from numpy's seeded generator, then
rounded to float16.  The float16 bits are the test input for both sides.

The shapes stand in for the networks the workloads are named after (an AlexNet conv pair,
the VGG-16 conv stack, MobileNet-v1 depthwise-separable blocks, the ResNet-50 convs) and
for the paper's own CNN benchmarks (Section 4); no dataset, network file or trained weight
is used anywhere.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


@dataclass(frozen=True)
class Layer:
    """One convolution layer (square kernel/stride/pad as in every listed workload)."""
    name: str
    c: int            # input channels
    h: int            # input plane (h == w)
    k: int            # output channels
    r: int            # kernel extent (r == s)
    stride: int = 1
    pad: int = 0
    dil: int = 1
    group: int = 1
    relu: bool = True
    out: int = 0      # output plane extent, written out by hand (checked in the tests)
    x_lo: float = 0.0  # inputs are uniform[x_lo, 1)
    count: int = 1    # how many times this exact shape occurs in the network

    def fan_in(self) -> int:
        return (self.c // self.group) * self.r * self.r


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    batch: int
    layers: List[Layer] = field(default_factory=list)

    def expanded(self) -> List[Layer]:
        """Layer list with repeated shapes unrolled (one entry per network layer)."""
        outl = []
        for l in self.layers:
            outl.extend([l] * l.count)
        return outl

    def expanded_unique(self) -> List[Layer]:
        """Distinct layer shapes in network order, `count` = how often each occurs."""
        import dataclasses
        seen = {}
        for l in self.expanded():
            key = (l.c, l.h, l.k, l.r, l.stride, l.pad, l.dil, l.group, l.relu)
            if key in seen:
                seen[key] = dataclasses.replace(seen[key], count=seen[key].count + 1)
            else:
                seen[key] = dataclasses.replace(l, count=1)
        return list(seen.values())


def _single() -> List[Layer]:
    return [Layer("conv3x3", 3, 32, 16, 3, 1, 1, out=32, x_lo=-1.0)]


def _alexnet_pair() -> List[Layer]:
    return [
        Layer("conv1", 3, 227, 96, 11, 4, 0, out=55, x_lo=-1.0),
        Layer("conv2", 96, 27, 256, 5, 1, 2, group=2, out=27, x_lo=-1.0),
    ]


def _vgg16() -> List[Layer]:
    spec = [("conv1_1", 3, 224, 64), ("conv1_2", 64, 224, 64),
            ("conv2_1", 64, 112, 128), ("conv2_2", 128, 112, 128),
            ("conv3_1", 128, 56, 256), ("conv3_2", 256, 56, 256), ("conv3_3", 256, 56, 256),
            ("conv4_1", 256, 28, 512), ("conv4_2", 512, 28, 512), ("conv4_3", 512, 28, 512),
            ("conv5_1", 512, 14, 512), ("conv5_2", 512, 14, 512), ("conv5_3", 512, 14, 512)]
    return [Layer(nm, c, h, k, 3, 1, 1, out=h) for nm, c, h, k in spec]


def _mobilenet_v1() -> List[Layer]:
    layers = [Layer("stem", 3, 224, 32, 3, 2, 1, out=112)]
    widths = [32, 64, 128, 128, 256, 256, 512, 512, 512, 512, 512, 512, 1024, 1024]
    plane = 112
    for i in range(1, 14):
        cin, cout = widths[i - 1], widths[i]
        s = 2 if i in (2, 4, 6, 12) else 1
        oplane = plane // s
        layers.append(Layer(f"dw{i}", cin, plane, cin, 3, s, 1, group=cin, out=oplane))
        layers.append(Layer(f"pw{i}", cin, oplane, cout, 1, 1, 0, out=oplane))
        plane = oplane
    return layers


def _resnet50() -> List[Layer]:
    layers = [Layer("stem", 3, 224, 64, 7, 2, 3, out=112)]
    cin = 64
    plane = 56
    for stage, (mid, cout, blocks) in enumerate(
            [(64, 256, 3), (128, 512, 4), (256, 1024, 6), (512, 2048, 3)], start=1):
        for b in range(1, blocks + 1):
            s = 2 if (stage > 1 and b == 1) else 1
            layers.append(Layer(f"s{stage}b{b}.a", cin, plane, mid, 1, 1, 0, out=plane))
            layers.append(Layer(f"s{stage}b{b}.b", mid, plane, mid, 3, s, 1, out=plane // s))
            plane //= s
            layers.append(Layer(f"s{stage}b{b}.c", mid, plane, cout, 1, 1, 0, relu=False, out=plane))
            cin = cout
    return layers


_BUILDERS = {0: ("single3x3", _single), 1: ("alexnet_pair", _alexnet_pair), 2: ("vgg16", _vgg16),
             3: ("mobilenet_v1", _mobilenet_v1), 4: ("resnet50", _resnet50)}
_BATCHES = {0: (1,), 1: (1,), 2: (1, 16), 3: (1, 32), 4: (64,)}


def workload(config_id: int, batch: Optional[int] = None) -> Workload:
    name, fn = _BUILDERS[config_id]
    if batch is None:
        batch = _BATCHES[config_id][-1]
    return Workload(f"{name}_n{batch}", config_id, batch, fn())


def all_workloads() -> List[Workload]:
    return [workload(c, b) for c in sorted(_BUILDERS) for b in _BATCHES[c]]


def by_name(name: str) -> Workload:
    for wl in all_workloads():
        if wl.name == name:
            return wl
    raise KeyError(f"unknown workload {name!r}; known: {[w.name for w in all_workloads()]}")


def make_tensors(config_id: int, batch: int, layer_index: int, layer: Layer, seed: int = 0,
                 batch_override: Optional[int] = None):
    """x [N,C,H,W], w [K,C/g,R,R], bias [K] as float16, drawn in that order from
    default_rng([seed, config_id, batch, layer_index]).  x ~ U[x_lo,1), w ~ N(0, std =
    sqrt(2/fan_in)) ("He-normal"), bias ~ U[-0.1,0.1).  batch_override keeps the stream's
    seed but draws fewer/more images (used for bounded samples of a large batch)."""
    rng = np.random.default_rng([seed, config_id, batch, layer_index])
    n = batch if batch_override is None else batch_override
    x = rng.uniform(layer.x_lo, 1.0, size=(n, layer.c, layer.h, layer.h)).astype(np.float16)
    std = float(np.sqrt(2.0 / layer.fan_in()))
    w = rng.normal(0.0, std, size=(layer.k, layer.c // layer.group, layer.r, layer.r)).astype(np.float16)
    b = rng.uniform(-0.1, 0.1, size=(layer.k,)).astype(np.float16)
    return x, w, b


def random_layer_tensors(rng: np.random.Generator, n, c, h, w, k, r, s, group):
    """Small random problem for property tests: x ~ U[-1,1), w ~ N(0, sqrt(2/fan_in))."""
    x = rng.uniform(-1.0, 1.0, size=(n, c, h, w)).astype(np.float16)
    std = float(np.sqrt(2.0 / max(1, (c // group) * r * s)))
    wt = rng.normal(0.0, std, size=(k, c // group, r, s)).astype(np.float16)
    b = rng.uniform(-0.1, 0.1, size=(k,)).astype(np.float16)
    return x, wt, b
