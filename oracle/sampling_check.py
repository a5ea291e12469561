"""Soundness of the oracle's bounds by sampling (TEST INFRASTRUCTURE, like the rest of oracle/).

A sound certifier's bounds enclose every concrete execution: for x in the input box, every pre-activation of every
layer lies in [lb, ub] (Section 2: the abstract shape over-approximates the neuron's values on the input region).
Concrete points are drawn from the box (half uniformly, half at random vertices, where the extremes of piecewise
linear functions tend to sit), pushed through the network in float64, and compared with the oracle's bounds.
The forward pass is the textbook one (matrix products, torch's conv2d): it shares nothing with the certifier.
"""
import numpy as np


def box(centers, eps, clip_lo, clip_hi):
    c = np.asarray(centers, dtype=np.float32)
    e = np.float32(eps)
    lo = np.maximum((c - e).astype(np.float32), np.float32(clip_lo)).astype(np.float64)
    hi = np.minimum((c + e).astype(np.float32), np.float32(clip_hi)).astype(np.float64)
    return lo, hi


def samples(l0, u0, m, rng):
    """m points of the box [l0, u0]: the first half uniform, the second half random vertices."""
    n = l0.shape[0]
    u = rng.random((m, n))
    x = l0 + (u0 - l0) * u
    half = m // 2
    x[half:] = np.where(u[half:] < 0.5, l0, u0)
    return x


def forward_preactivations(layers, x):
    """Float64 forward pass; x [m, n0]; returns [m, n_total] pre-activations of every affine layer."""
    import torch
    a = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64))
    outs = []
    for l in layers:
        w = torch.from_numpy(np.asarray(l.weight, dtype=np.float64))
        b = torch.from_numpy(np.asarray(l.bias, dtype=np.float64))
        if l.kind == "fc":
            z = a.reshape(a.shape[0], -1) @ w.T + b
        else:
            z = torch.nn.functional.conv2d(a.reshape(a.shape[0], *l.in_shape), w, b, stride=l.stride, padding=l.pad)
            z = z.reshape(z.shape[0], -1)
        outs.append(z)
        a = torch.clamp(z, min=0.0) if l.relu_after else z
    return torch.cat(outs, dim=1).numpy()


def check_box(layers, lb, ub, l0, u0, m, seed, chunk=10000):
    """Violations of lb - d <= z <= ub + d, d = 1e-9 * (1 + |bound|), over m samples of one box.
    Returns (violations, smallest slack: min over samples and neurons of min(z - lb, ub - z))."""
    rng = np.random.default_rng(seed)
    viol, slack = 0, np.inf
    dl, du = 1e-9 * (1 + np.abs(lb)), 1e-9 * (1 + np.abs(ub))
    for start in range(0, m, chunk):
        z = forward_preactivations(layers, samples(l0, u0, min(chunk, m - start), rng))
        viol += int((z < lb - dl).sum() + (z > ub + du).sum())
        slack = min(slack, float((z - lb).min()), float((ub - z).min()))
    return viol, slack
