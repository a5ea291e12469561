"""Pins for residual connections in the oracle.  The paper lists a residual network among its benchmarks
(Appendix, table of DNNs: "Skip") and its DeepPoly listing covers it without change: the neuron of a layer
with a connection is an Affine neuron whose prev holds neurons of two layers, and traverse (priority
-layer) replaces the neurons of the highest layer first.  Pinned here by a hand-worked example, by the
closed form of a net without ReLUs, by the forward pass at eps = 0, by sampling, by brute force, and by a
second, layer-level implementation."""
import json
import os

import numpy as np
import pytest

from oracle import deeppoly_oracle as orc
from oracle import deeppoly_matrix_np as mat
from paper_2507_20055_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _forward(w, x):
    """Pre-activations of every affine layer for inputs x [m, n0], float64, with the residual connections."""
    A = [mat.dense_matrix(l) for l in w.layers]
    bias = [mat.dense_bias(l) for l in w.layers]
    acts, zs, a = [], [], np.asarray(x, np.float64)
    for k, l in enumerate(w.layers):
        z = a @ A[k].T + bias[k]
        if w.skip_from is not None and w.skip_from[k] >= 0:
            z = z + acts[w.skip_from[k]]
        zs.append(z)
        a = np.maximum(z, 0.0) if l.relu_after else z
        acts.append(a)
    return np.concatenate(zs, axis=1)


def test_hand_worked_residual_example():
    g = json.load(open(os.path.join(GOLD, "residual_example.json")))
    layers = [wl.Layer("fc", np.array(l["weight"], np.float32), np.array(l["bias"], np.float32),
                       relu_after=l["relu_after"]) for l in g["layers"]]
    c = np.array([g["center"]], np.float32)
    r = orc.deeppoly(layers, c, g["eps"], *g["clip"], skip_from=g["skip_from"])
    np.testing.assert_allclose(r["lb"][0], g["lb"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(r["ub"][0], g["ub"], rtol=0, atol=1e-15)
    assert r["codes"][0].tolist() == g["codes"]
    lb, ub, codes = mat.deeppoly_matrix(layers, c, g["eps"], *g["clip"], skip_from=g["skip_from"])
    np.testing.assert_allclose(lb[0], g["lb"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(ub[0], g["ub"], rtol=0, atol=1e-15)
    # without the connection the last neuron is -a1 alone: [-1, 1] by the same rules (lower -0.75x - 0.25,
    # upper -2x + 1), so the example does tell
    plain = orc.deeppoly(layers, c, g["eps"], *g["clip"])
    assert plain["lb"][0, 2] == pytest.approx(-1.0) and plain["ub"][0, 2] == pytest.approx(1.0)


def test_closed_form_without_relus():
    w = wl.residual_fc(6, 7, 2, 3, batch=3, eps=0.07, seed=11)
    for l in w.layers:
        l.relu_after = False
    # a_k = M_k x + c_k with M_k = W_k M_{k-1} + M_s, c_k = W_k c_{k-1} + b_k + c_s
    Ms, cs, lbs, ubs = [], [], [], []
    l0, u0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    M, c = np.eye(6), np.zeros(6)
    for k, l in enumerate(w.layers):
        W, b = l.weight.astype(np.float64), l.bias.astype(np.float64)
        M, c = W @ M, W @ c + b
        s = w.skip_from[k]
        if s >= 0:
            M, c = M + Ms[s], c + cs[s]
        Ms.append(M); cs.append(c)
        lbs.append(l0 @ np.clip(M, 0, None).T + u0 @ np.clip(M, None, 0).T + c)
        ubs.append(u0 @ np.clip(M, 0, None).T + l0 @ np.clip(M, None, 0).T + c)
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    np.testing.assert_allclose(r["lb"], np.concatenate(lbs, axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(r["ub"], np.concatenate(ubs, axis=1), rtol=0, atol=1e-12)


@pytest.mark.parametrize("kind", ["fc", "conv"])
def test_eps_zero_is_the_forward_pass(kind):
    w = wl.residual_fc(8, 10, 2, 4, batch=4, eps=0.0, seed=12) if kind == "fc" else \
        wl.residual_conv((2, 6, 6), 3, 1, 4, batch=2, eps=0.0, seed=13)
    r = orc.deeppoly(w.layers, w.centers, 0.0, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    z = _forward(w, w.centers)
    np.testing.assert_allclose(r["lb"], z, rtol=0, atol=1e-12)
    np.testing.assert_allclose(r["ub"], z, rtol=0, atol=1e-12)


@pytest.mark.parametrize("kind", ["fc", "conv"])
def test_sound_by_sampling_and_connection_matters(kind):
    w = wl.residual_fc(8, 12, 2, 4, batch=3, eps=0.05, seed=14) if kind == "fc" else \
        wl.residual_conv((2, 6, 6), 3, 2, 4, batch=2, eps=0.03, seed=15)
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    l0, u0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    rng = np.random.default_rng(5)
    for b in range(w.batch):
        u = rng.random((4000, l0.shape[1]))
        u[2000:] = (u[2000:] > 0.5)                      # half of the samples are vertices
        x = l0[b] + u * (u0[b] - l0[b])
        z = _forward(w, x)
        tol = 1e-9 * (1 + np.abs(z))
        assert (z >= r["lb"][b] - tol).all() and (z <= r["ub"][b] + tol).all()
    assert (r["lb"] <= r["ub"]).all()
    plain = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    assert np.abs(plain["lb"] - r["lb"]).max() > 1e-3    # a net without the connections is another net


@pytest.mark.parametrize("kind", ["fc", "conv"])
def test_agrees_with_the_layer_level_form(kind):
    w = wl.residual_fc(9, 11, 3, 5, batch=3, eps=0.04, seed=16) if kind == "fc" else \
        wl.residual_conv((2, 8, 6), 4, 2, 3, batch=2, eps=0.02, seed=17)
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    lb, ub, codes = mat.deeppoly_matrix(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    np.testing.assert_allclose(r["lb"], lb, rtol=0, atol=1e-10)
    np.testing.assert_allclose(r["ub"], ub, rtol=0, atol=1e-10)
    assert (r["codes"] == codes).all()


def test_brute_force_on_a_tiny_net():
    w = wl.residual_fc(2, 3, 1, 2, batch=1, eps=0.3, seed=18)
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    l0, u0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    g = np.linspace(0.0, 1.0, 1001)
    xx, yy = np.meshgrid(g, g, indexing="ij")
    x = np.stack([l0[0, 0] + xx.ravel() * (u0[0, 0] - l0[0, 0]), l0[0, 1] + yy.ravel() * (u0[0, 1] - l0[0, 1])], axis=1)
    z = _forward(w, x)
    assert (z.min(axis=0) >= r["lb"][0] - 1e-9).all() and (z.max(axis=0) <= r["ub"][0] + 1e-9).all()
    # the first layer is exact (an interval of an affine map)
    np.testing.assert_allclose(z.min(axis=0)[:3], r["lb"][0][:3], atol=1e-9)


def test_malformed_connections_are_refused():
    w = wl.residual_fc(4, 5, 1, 2, batch=1, eps=0.1, seed=19)
    with pytest.raises(RuntimeError):
        orc.deeppoly(w.layers, w.centers, w.eps, skip_from=[-1, 0, -1, -1])        # not two layers back
    with pytest.raises(RuntimeError):
        orc.deeppoly(w.layers, w.centers, w.eps, skip_from=[-1, -1, -1, 1])        # widths differ
    with pytest.raises(RuntimeError):
        orc.deeppoly(w.layers, w.centers, w.eps, skip_from=w.skip_from, skip_form=True)


# ---- traversals that stop early (DeepPoly_p, IBP, CROWN-IBP) with a connection still open ----

def test_hand_worked_example_early_stops():
    g = json.load(open(os.path.join(GOLD, "residual_example.json")))
    layers = [wl.Layer("fc", np.array(l["weight"], np.float32), np.array(l["bias"], np.float32),
                       relu_after=l["relu_after"]) for l in g["layers"]]
    c = np.array([g["center"]], np.float32)
    runs = {"ibp": dict(backsteps_per_layer=[0, 0, 0]), "deeppoly_p1": dict(max_backsteps=1)}
    for name, kw in runs.items():
        v = g["variants"][name]
        r = orc.deeppoly(layers, c, g["eps"], *g["clip"], skip_from=g["skip_from"], **kw)
        np.testing.assert_allclose(r["lb"][0], v["lb"], rtol=0, atol=1e-15, err_msg=name)
        np.testing.assert_allclose(r["ub"][0], v["ub"], rtol=0, atol=1e-15, err_msg=name)
        assert r["codes"][0].tolist() == v["codes"], name
        steps = kw.get("backsteps_per_layer", [1, 1, 1])
        lb, ub, _ = mat.deeppoly_matrix(layers, c, g["eps"], *g["clip"], skip_from=g["skip_from"], backsteps=steps)
        np.testing.assert_allclose(lb[0], v["lb"], rtol=0, atol=1e-15, err_msg=name)
        np.testing.assert_allclose(ub[0], v["ub"], rtol=0, atol=1e-15, err_msg=name)


def test_ibp_is_interval_arithmetic_with_the_connections():
    w = wl.residual_fc(7, 9, 2, 3, batch=3, eps=0.05, seed=31)
    r = orc.ibp(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    l, u = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    acts, off = [], 0
    for k, layer in enumerate(w.layers):
        W, b = layer.weight.astype(np.float64), layer.bias.astype(np.float64)
        lo = l @ np.clip(W, 0, None).T + u @ np.clip(W, None, 0).T + b
        up = u @ np.clip(W, 0, None).T + l @ np.clip(W, None, 0).T + b
        if w.skip_from[k] >= 0:
            lo, up = lo + acts[w.skip_from[k]][0], up + acts[w.skip_from[k]][1]
        n = W.shape[0]
        np.testing.assert_allclose(r["lb"][:, off:off + n], lo, rtol=0, atol=1e-12)
        np.testing.assert_allclose(r["ub"][:, off:off + n], up, rtol=0, atol=1e-12)
        off += n
        l, u = (np.maximum(lo, 0), np.maximum(up, 0)) if layer.relu_after else (lo, up)
        acts.append((l, u))


@pytest.mark.parametrize("kind", ["fc", "conv"])
def test_early_stops_sound_and_agree_with_the_layer_level_form(kind):
    w = wl.residual_fc(8, 12, 2, 4, batch=3, eps=0.05, seed=32) if kind == "fc" else \
        wl.residual_conv((2, 6, 6), 3, 2, 4, batch=2, eps=0.03, seed=33)
    K = len(w.layers)
    l0, u0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    rng = np.random.default_rng(6)
    full = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    for name, steps in {"ibp": [0] * K, "crown_ibp": [0] * (K - 1) + [-1], "p1": [1] * K, "p2": [2] * K,
                        "p3": [3] * K, "mixed": [(-1 if k % 2 else 1) for k in range(K)]}.items():
        r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                         backsteps_per_layer=steps)
        lb, ub, codes = mat.deeppoly_matrix(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                                            backsteps=steps)
        np.testing.assert_allclose(r["lb"], lb, rtol=0, atol=1e-10, err_msg=name)
        np.testing.assert_allclose(r["ub"], ub, rtol=0, atol=1e-10, err_msg=name)
        for b in range(w.batch):
            uu = rng.random((2000, l0.shape[1]))
            uu[1000:] = (uu[1000:] > 0.5)
            z = _forward(w, l0[b] + uu * (u0[b] - l0[b]))
            tol = 1e-9 * (1 + np.abs(z))
            assert (z >= r["lb"][b] - tol).all() and (z <= r["ub"][b] + tol).all(), name
    # as many steps as there are layers is the full traversal
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from, max_backsteps=K)
    np.testing.assert_allclose(r["lb"], full["lb"], rtol=0, atol=1e-13)
