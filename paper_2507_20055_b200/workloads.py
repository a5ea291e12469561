"""Seeded synthetic networks and input boxes (no certifier arithmetic here).

The paper evaluates on trained MNIST / CIFAR10 networks (Appendix, table of
32 DNNs); those weights and images are not available, so networks with the
same layer shapes and random weights stand in for them.  This module only
draws numbers: both the CPU oracle and the CUDA library are fed from the
arrays made here, and neither is imported here.

Generator: a counter-based stream.  Word i of stream (seed, stream_id) is
splitmix64(seed * 2^32 + stream_id, i); uniforms take the top 53 bits;
normals are Box-Muller pairs in float64, rounded once to float32.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        return z ^ (z >> np.uint64(31))


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    """n float64 uniforms in [0,1) from stream (seed, stream)."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(seed << 32) ^ stream], dtype=np.uint64))[0]
        ctr = np.arange(n, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15) + key
    bits = _splitmix64(ctr)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """n float64 standard normals (Box-Muller on consecutive uniform pairs)."""
    m = (n + 1) // 2
    u = uniform01(seed, stream, 2 * m)
    u1 = 1.0 - u[0::2]          # (0,1]
    u2 = u[1::2]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * m, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n]


@dataclass
class Layer:
    """One affine layer, optionally followed by a ReLU layer.

    kind 'fc':   weight [out, in]               float32
    kind 'conv': weight [c_out, c_in, kh, kw]   float32, in_shape = (c_in, h, w)
    """
    kind: str
    weight: np.ndarray
    bias: np.ndarray
    relu_after: bool = True
    stride: int = 1
    pad: int = 0
    in_shape: Optional[Tuple[int, int, int]] = None

    @property
    def n_in(self) -> int:
        if self.kind == "fc":
            return int(self.weight.shape[1])
        c, h, w = self.in_shape
        return c * h * w

    @property
    def out_shape(self) -> Tuple[int, int, int]:
        c, h, w = self.in_shape
        co, _, kh, kw = self.weight.shape
        return (co, (h + 2 * self.pad - kh) // self.stride + 1,
                (w + 2 * self.pad - kw) // self.stride + 1)

    @property
    def n_out(self) -> int:
        if self.kind == "fc":
            return int(self.weight.shape[0])
        co, ho, wo = self.out_shape
        return co * ho * wo


@dataclass
class Workload:
    name: str
    layers: List[Layer]
    centers: np.ndarray          # [batch, n0] float32
    eps: float
    clip_lo: float = 0.0
    clip_hi: float = 1.0
    notes: dict = field(default_factory=dict)
    # residual connections: skip_from[k] = s >= 0 adds the outputs of layer s to layer k's affine result
    # (equal widths, s <= k-2); None or -1 = none
    skip_from: Optional[List[int]] = None

    @property
    def batch(self) -> int:
        return int(self.centers.shape[0])

    @property
    def n_total(self) -> int:
        return sum(l.n_out for l in self.layers)

    @property
    def n_relu(self) -> int:
        return sum(l.n_out for l in self.layers if l.relu_after)


def fc_net(sizes, seed=0, stream0=0, w_sigma="fan_in", b_sigma=0.1, relu_last=False) -> List[Layer]:
    """FC ReLU net; weights N(0, 1/fan_in) (sigma = fan_in^-1/2), biases N(0, 0.01) (sigma 0.1)."""
    layers = []
    for k in range(len(sizes) - 1):
        n_in, n_out = sizes[k], sizes[k + 1]
        sw = n_in ** -0.5 if w_sigma == "fan_in" else float(w_sigma)
        w = (normal(seed, stream0 + 2 * k, n_out * n_in) * sw).astype(np.float32).reshape(n_out, n_in)
        b = (normal(seed, stream0 + 2 * k + 1, n_out) * b_sigma).astype(np.float32)
        layers.append(Layer("fc", w, b, relu_after=(k < len(sizes) - 2) or relu_last))
    return layers


def conv_layer(in_shape, c_out, k, stride, pad, seed, stream, b_sigma=0.1, relu_after=True) -> Layer:
    """He-normal conv layer: sigma = sqrt(2 / (c_in*k*k))."""
    c_in = in_shape[0]
    sw = (2.0 / (c_in * k * k)) ** 0.5
    w = (normal(seed, stream, c_out * c_in * k * k) * sw).astype(np.float32).reshape(c_out, c_in, k, k)
    b = (normal(seed, stream + 1, c_out) * b_sigma).astype(np.float32)
    return Layer("conv", w, b, relu_after=relu_after, stride=stride, pad=pad, in_shape=tuple(in_shape))


def centers_uniform(batch, n0, seed=0, stream=1000) -> np.ndarray:
    return uniform01(seed, stream, batch * n0).astype(np.float32).reshape(batch, n0)


# The five benchmark configurations (index 0..4).
CONFIG_NAMES = ["fc3x50_b1", "fc6x100_b64", "fc9x200_b256", "convsmall_b32", "fc6x1024_b128"]


def make_config(idx: int, seed: int = 0, batch: Optional[int] = None) -> Workload:
    """Configuration idx (0-based) of the benchmark list, seeded."""
    if idx == 0:
        sizes, b, eps = [784, 50, 50, 50, 10], 1, 0.01
    elif idx == 1:
        sizes, b, eps = [784] + [100] * 6 + [10], 64, 0.02
    elif idx == 2:
        sizes, b, eps = [784] + [200] * 9 + [10], 256, 0.015
    elif idx == 4:
        sizes, b, eps = [784] + [1024] * 6 + [10], 128, 0.01
    elif idx == 3:
        b, eps = 32, 2.0 / 255.0
        if batch is not None:
            b = batch
        l1 = conv_layer((3, 32, 32), 16, 4, 2, 1, seed, 0)
        l2 = conv_layer(l1.out_shape, 32, 4, 2, 1, seed, 2)
        n2 = l2.n_out
        sw3, sw4 = (2.0 / n2) ** 0.5, (2.0 / 100) ** 0.5
        fcs = []
        for k, (n_in, n_out, sw) in enumerate([(n2, 100, sw3), (100, 10, sw4)]):
            w = (normal(seed, 4 + 2 * k, n_out * n_in) * sw).astype(np.float32).reshape(n_out, n_in)
            bb = (normal(seed, 5 + 2 * k, n_out) * 0.1).astype(np.float32)
            fcs.append(Layer("fc", w, bb, relu_after=(k == 0)))
        layers = [l1, l2] + fcs
        return Workload(CONFIG_NAMES[idx], layers, centers_uniform(b, 3 * 32 * 32, seed), eps)
    else:
        raise ValueError(f"no config {idx}")
    if batch is not None:
        b = batch
    return Workload(CONFIG_NAMES[idx], fc_net(sizes, seed), centers_uniform(b, sizes[0], seed), eps)


def small_fc(sizes, batch, eps, seed=1, relu_last=False, b_sigma=0.1, clip=(0.0, 1.0)) -> Workload:
    layers = fc_net(sizes, seed, relu_last=relu_last, b_sigma=b_sigma)
    return Workload("fc_" + "x".join(map(str, sizes)), layers, centers_uniform(batch, sizes[0], seed),
                    eps, clip[0], clip[1])


def small_conv(in_shape, convs, fcs, batch, eps, seed=2) -> Workload:
    """convs: list of (c_out, k, stride, pad); fcs: list of widths after flatten."""
    layers, shape, stream = [], tuple(in_shape), 0
    for (co, k, s, p) in convs:
        l = conv_layer(shape, co, k, s, p, seed, stream)
        layers.append(l)
        shape, stream = l.out_shape, stream + 2
    n = shape[0] * shape[1] * shape[2]
    for i, wdt in enumerate(fcs):
        w = (normal(seed, stream, wdt * n) * (2.0 / n) ** 0.5).astype(np.float32).reshape(wdt, n)
        bb = (normal(seed, stream + 1, wdt) * 0.1).astype(np.float32)
        layers.append(Layer("fc", w, bb, relu_after=(i < len(fcs) - 1)))
        n, stream = wdt, stream + 2
    if not fcs:
        layers[-1].relu_after = False
    n0 = in_shape[0] * in_shape[1] * in_shape[2]
    return Workload("conv_small", layers, centers_uniform(batch, n0, seed), eps)


def residual_fc(n0, width, blocks, n_out, batch, eps, seed=3) -> Workload:
    """x -> FC(width)+ReLU -> blocks x [FC(width)+ReLU -> FC(width) (+ block input) + ReLU] -> FC(n_out):
    a fully connected residual net in the shape of the paper's "Skip" network (Appendix, table of DNNs)."""
    sizes = [n0, width] + [width] * (2 * blocks) + [n_out]
    layers = fc_net(sizes, seed)
    skip = [-1] * len(layers)
    for b in range(blocks):
        skip[2 + 2 * b] = 2 * b          # the block's second layer adds the block's input (outputs of layer 2b)
    return Workload(f"resfc_{n0}_{width}x{blocks}", layers, centers_uniform(batch, n0, seed), eps, skip_from=skip)


def residual_conv(in_shape, c, blocks, n_out, batch, eps, seed=4) -> Workload:
    """conv(c, 3x3, s2, p1)+ReLU -> blocks x [conv(c,3x3,s1,p1)+ReLU -> conv(c,3x3,s1,p1) (+ block input) + ReLU]
    -> FC(n_out)."""
    layers, stream = [], 0
    l = conv_layer(tuple(in_shape), c, 3, 2, 1, seed, stream)
    layers.append(l)
    shape, stream = l.out_shape, stream + 2
    skip = [-1]
    for b in range(blocks):
        for half in range(2):
            l = conv_layer(shape, c, 3, 1, 1, seed, stream)
            layers.append(l)
            shape, stream = l.out_shape, stream + 2
            skip.append(2 * b if half == 1 else -1)
    n = shape[0] * shape[1] * shape[2]
    w = (normal(seed, stream, n_out * n) * (2.0 / n) ** 0.5).astype(np.float32).reshape(n_out, n)
    bb = (normal(seed, stream + 1, n_out) * 0.1).astype(np.float32)
    layers.append(Layer("fc", w, bb, relu_after=False))
    skip.append(-1)
    n0 = in_shape[0] * in_shape[1] * in_shape[2]
    return Workload("resconv", layers, centers_uniform(batch, n0, seed), eps, skip_from=skip)
