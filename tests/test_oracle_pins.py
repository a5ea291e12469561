"""Pins for the float64 oracle: everything here is fixed by the paper's DeepPoly
specification (Appendix C) or by mathematics, not by the oracle itself."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import deeppoly_oracle as orc
from oracle import deeppoly_matrix_np as mat
from paper_2507_20055_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _fr(xs):
    return np.array([float(Fraction(x)) for x in xs])


def _w1(bias1=None):
    g = json.load(open(os.path.join(GOLD, "w1_example.json")))
    layers = []
    for l in g["layers"]:
        layers.append(wl.Layer("fc", np.array(l["weight"], np.float32), np.array(l["bias"], np.float32),
                               relu_after=l["relu_after"]))
    if bias1 is not None:
        layers[0].bias = np.array(bias1, np.float32)
    return g, layers


def test_w1_worked_example():
    g, layers = _w1()
    r = orc.deeppoly(layers, np.array([g["center"]], np.float32), g["eps"], *g["clip"])
    np.testing.assert_allclose(r["lb"][0], _fr(g["lb"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(r["ub"][0], _fr(g["ub"]), rtol=0, atol=1e-14)
    assert r["codes"][0].tolist() == g["codes"]


def test_w1_batch_independence():
    g, layers = _w1()
    c = np.array([g["center"], g["center"], [0.25, 0.75]], np.float32)
    r = orc.deeppoly(layers, c, g["eps"], *g["clip"])
    assert np.array_equal(r["lb"][0], r["lb"][1]) and np.array_equal(r["ub"][0], r["ub"][1])
    r2 = orc.deeppoly(layers, c[2:], g["eps"], *g["clip"])
    assert np.array_equal(r["lb"][2], r2["lb"][0]) and np.array_equal(r["ub"][2], r2["ub"][0])


@pytest.mark.parametrize("fp32", [True, False])
def test_w1_tie_rule(fp32):
    g, layers = _w1(bias1=[0.0, 0.0])
    t = g["tie_variant"]
    r = orc.deeppoly(layers, np.zeros((1, 2), np.float32), 1.0, -1.0, 1.0, decision_fp32=fp32)
    np.testing.assert_allclose(r["lb"][0, :2], _fr(t["lb_layer1"]), atol=0)
    np.testing.assert_allclose(r["ub"][0, :2], _fr(t["ub_layer1"]), atol=0)
    assert r["codes"][0, :2].tolist() == t["codes_layer1"]
    np.testing.assert_allclose(r["lb"][0, 2:4], _fr(t["lb_layer2"]), atol=1e-15)
    np.testing.assert_allclose(r["ub"][0, 2:4], _fr(t["ub_layer2"]), atol=1e-15)


def _linear_closed_form(layers, l0, u0):
    """Exact min/max of every prefix of an all-linear net over a box."""
    A, c = None, None
    lbs, ubs = [], []
    for l in layers:
        W, b = mat.dense_matrix(l), mat.dense_bias(l)
        A, c = (W, b) if A is None else (W @ A, W @ c + b)
        Ap, Am = np.maximum(A, 0), np.minimum(A, 0)
        lbs.append(Ap @ l0 + Am @ u0 + c)
        ubs.append(Ap @ u0 + Am @ l0 + c)
    return np.concatenate(lbs), np.concatenate(ubs)


def test_all_linear_network_is_exact():
    w = wl.small_fc([7, 9, 5, 6, 3], batch=3, eps=0.1, seed=11)
    for l in w.layers:
        l.relu_after = False
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    L0, U0 = mat.box(w.centers, w.eps, 0.0, 1.0)
    for b in range(w.batch):
        lb, ub = _linear_closed_form(w.layers, L0[b], U0[b])
        np.testing.assert_allclose(r["lb"][b], lb, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(r["ub"][b], ub, rtol=1e-12, atol=1e-12)
    assert r["codes"].shape[1] == 0


def test_all_linear_conv_network_is_exact():
    w = wl.small_conv((2, 7, 6), [(3, 3, 2, 1), (4, 2, 1, 0)], [5, 3], batch=2, eps=0.05, seed=5)
    for l in w.layers:
        l.relu_after = False
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    L0, U0 = mat.box(w.centers, w.eps, 0.0, 1.0)
    for b in range(w.batch):
        lb, ub = _linear_closed_form(w.layers, L0[b], U0[b])
        np.testing.assert_allclose(r["lb"][b], lb, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(r["ub"][b], ub, rtol=1e-12, atol=1e-12)


def test_eps_zero_is_the_forward_pass_fc():
    w = wl.small_fc([12, 20, 20, 20, 4], batch=4, eps=0.0, seed=3)
    r = orc.deeppoly(w.layers, w.centers, 0.0)
    z = mat.forward_preactivations(w.layers, w.centers)
    np.testing.assert_allclose(r["lb"], z, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(r["ub"], z, rtol=1e-12, atol=1e-12)
    assert set(np.unique(r["codes"])) <= {0, 1}


def test_eps_zero_conv_matches_torch_conv2d():
    """Pins conv geometry (stride, padding, cross-correlation, (c,h,w) flattening)
    to a library routine."""
    torch = pytest.importorskip("torch")
    w = wl.small_conv((3, 9, 8), [(4, 4, 2, 1), (5, 3, 1, 1)], [6, 3], batch=3, eps=0.0, seed=9)
    r = orc.deeppoly(w.layers, w.centers, 0.0)
    x = torch.tensor(w.centers, dtype=torch.float64).reshape(3, 3, 9, 8)
    outs = []
    a = x
    for l in w.layers:
        W = torch.tensor(l.weight, dtype=torch.float64)
        bb = torch.tensor(l.bias, dtype=torch.float64)
        if l.kind == "conv":
            z = torch.nn.functional.conv2d(a, W, bb, stride=l.stride, padding=l.pad)
        else:
            z = a.reshape(3, -1) @ W.T + bb
        outs.append(z.reshape(3, -1))
        a = torch.relu(z) if l.relu_after else z
    z = torch.cat(outs, dim=1).numpy()
    np.testing.assert_allclose(r["lb"], z, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(r["ub"], z, rtol=1e-12, atol=1e-12)


def test_all_stable_neurons_are_relaxed_exactly():
    """With large biases every hidden neuron is stable, so the net is linear on the
    box with the activation pattern fixed, and DeepPoly must be exact."""
    w = wl.small_fc([6, 8, 8, 3], batch=2, eps=0.02, seed=4, b_sigma=5.0)
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    assert set(np.unique(r["codes"])) <= {0, 1} and len(np.unique(r["codes"])) == 2
    L0, U0 = mat.box(w.centers, w.eps, 0.0, 1.0)
    for b in range(w.batch):
        codes = r["codes"][b]
        lin, off = [], 0
        for l in w.layers:
            W, bias = mat.dense_matrix(l).copy(), mat.dense_bias(l).copy()
            lin.append(wl.Layer("fc", W, bias, relu_after=False))
        # fold the fixed activation pattern into the next layer's columns
        off = 0
        for k, l in enumerate(w.layers[:-1]):
            n = l.n_out
            lin[k + 1].weight = lin[k + 1].weight * codes[off:off + n].astype(np.float64)
            off += n
        lb, ub = _linear_closed_form(lin, L0[b], U0[b])
        np.testing.assert_allclose(r["lb"][b], lb, rtol=1e-11, atol=1e-11)
        np.testing.assert_allclose(r["ub"][b], ub, rtol=1e-11, atol=1e-11)


def test_one_hidden_layer_closed_form():
    """lb_2 = min over the box of (W2+ lamL + W2- lamU)(W1 x + b1) + W2- nu + b2."""
    w = wl.small_fc([5, 16, 4], batch=3, eps=0.2, seed=8)
    r = orc.deeppoly(w.layers, w.centers, w.eps, decision_fp32=False)
    W1, b1 = w.layers[0].weight.astype(np.float64), w.layers[0].bias.astype(np.float64)
    W2, b2 = w.layers[1].weight.astype(np.float64), w.layers[1].bias.astype(np.float64)
    L0, U0 = mat.box(w.centers, w.eps, 0.0, 1.0)
    n_unstable = 0
    for b in range(w.batch):
        l0, u0 = L0[b], U0[b]
        l1 = np.maximum(W1, 0) @ l0 + np.minimum(W1, 0) @ u0 + b1
        u1 = np.maximum(W1, 0) @ u0 + np.minimum(W1, 0) @ l0 + b1
        lamL = (l1 + u1 >= 0).astype(float)
        lamU = np.where(l1 >= 0, 1.0, np.where(u1 <= 0, 0.0, u1 / (u1 - l1)))
        nu = np.where((l1 < 0) & (u1 > 0), -u1 * l1 / (u1 - l1), 0.0)
        n_unstable += int(((l1 < 0) & (u1 > 0)).sum())
        W2p, W2m = np.maximum(W2, 0), np.minimum(W2, 0)
        El = (W2p * lamL + W2m * lamU)
        Eu = (W2p * lamU + W2m * lamL)
        Cl, dl = El @ W1, El @ b1 + W2m @ nu + b2
        Cu, du = Eu @ W1, Eu @ b1 + W2p @ nu + b2
        lb2 = np.maximum(Cl, 0) @ l0 + np.minimum(Cl, 0) @ u0 + dl
        ub2 = np.maximum(Cu, 0) @ u0 + np.minimum(Cu, 0) @ l0 + du
        np.testing.assert_allclose(r["lb"][b], np.concatenate([l1, lb2]), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(r["ub"][b], np.concatenate([u1, ub2]), rtol=1e-12, atol=1e-12)
    assert n_unstable > 5


@pytest.mark.parametrize("make", [
    lambda: wl.small_fc([10, 24, 24, 24, 5], batch=3, eps=0.05, seed=21),
    lambda: wl.small_conv((2, 8, 8), [(4, 4, 2, 1), (6, 4, 2, 1)], [12, 4], batch=2, eps=0.03, seed=22),
    lambda: wl.small_conv((1, 7, 5), [(3, 3, 1, 0)], [4], batch=2, eps=0.1, seed=23),
    lambda: wl.make_config(0),
])
def test_matrix_form_agrees(make):
    w = make()
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    lb, ub, codes = mat.deeppoly_matrix(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(r["lb"], lb, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(r["ub"], ub, rtol=1e-10, atol=1e-10)
    assert np.array_equal(r["codes"], codes)
    assert (r["codes"] >= 2).sum() > 0


def _samples(l0, u0, m, seed):
    n = l0.shape[0]
    u = wl.uniform01(seed, 77, m * n).reshape(m, n)
    half = m // 2
    x = l0 + (u0 - l0) * u
    x[half:] = np.where(u[half:] < 0.5, l0, u0)          # random vertices
    return x


@pytest.mark.parametrize("make,m", [
    (lambda: wl.small_fc([8, 16, 16, 16, 4], batch=2, eps=0.1, seed=31), 100_000),
    (lambda: wl.small_conv((2, 6, 6), [(3, 4, 2, 1), (4, 2, 1, 0)], [8, 3], batch=1, eps=0.05, seed=32), 100_000),
    (lambda: wl.make_config(0), 100_000),
    (lambda: wl.make_config(1, batch=2), 20_000),
])
def test_soundness_by_sampling(make, m):
    w = make()
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    L0, U0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    for b in range(w.batch):
        z = mat.forward_preactivations(w.layers, _samples(L0[b], U0[b], m, seed=b))
        lb, ub = r["lb"][b], r["ub"][b]
        assert (z.min(axis=0) >= lb - 1e-9 * (1 + np.abs(lb))).all()
        assert (z.max(axis=0) <= ub + 1e-9 * (1 + np.abs(ub))).all()


def test_sampling_verdicts_of_the_large_configurations():
    """10^5 samples from every box of the three large configurations take tens of minutes: that run is made once by
    tests/golden/make_sampling_verdicts.py and its verdict stored; here the stored verdict is checked (no violation,
    every box, the oracle source it was made with is the current one) and the check repeated on a subsample."""
    import hashlib
    import json
    import os
    from oracle import sampling_check as sc
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    verdicts = json.load(open(os.path.join(root, "tests", "golden", "sampling_verdicts.json")))
    with open(os.path.join(root, "oracle", "deeppoly_oracle.c"), "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()[:16]
    for idx, boxes, m in ((2, 4, 5000), (3, 2, 5000), (4, 2, 2000)):
        w = wl.make_config(idx)
        v = verdicts[w.name]
        assert v["violations"] == 0 and v["samples_per_box"] == 100_000 and v["boxes"] == w.batch
        assert v["oracle_source_sha256_16"] == sha, "the oracle changed: run tests/golden/make_sampling_verdicts.py again"
        c = w.centers[:boxes]
        r = orc.deeppoly(w.layers, c, w.eps, w.clip_lo, w.clip_hi)
        l0, u0 = sc.box(c, w.eps, w.clip_lo, w.clip_hi)
        for b in range(boxes):
            viol, slack = sc.check_box(w.layers, r["lb"][b], r["ub"][b], l0[b], u0[b], m, seed=7 + b)
            assert viol == 0 and slack > -1e-6


def test_invariants_order_and_relaxation_ranges():
    w = wl.make_config(1, batch=3)
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    assert (r["lb"] <= r["ub"]).all()
    frac_unstable = (r["codes"] >= 2).mean()
    assert 0.05 < frac_unstable < 0.9


def test_permutation_and_scaling_invariance():
    w = wl.small_fc([6, 10, 10, 4], batch=2, eps=0.1, seed=41)
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    perm = np.array([3, 1, 4, 0, 9, 2, 7, 5, 8, 6])
    l = [wl.Layer("fc", x.weight.copy(), x.bias.copy(), x.relu_after) for x in w.layers]
    l[0].weight, l[0].bias = l[0].weight[perm], l[0].bias[perm]
    l[1].weight = l[1].weight[:, perm]
    scale = np.array([2.0, -4.0, 0.5, -1.0], dtype=np.float32)
    l[2].weight, l[2].bias = l[2].weight * scale[:, None], l[2].bias * scale
    r2 = orc.deeppoly(l, w.centers, w.eps)
    np.testing.assert_allclose(r2["lb"][:, :10], r["lb"][:, :10][:, perm], rtol=1e-12)
    np.testing.assert_allclose(r2["ub"][:, 10:20], r["ub"][:, 10:20], rtol=1e-12, atol=1e-13)
    lo, hi = r["lb"][:, 20:], r["ub"][:, 20:]
    exp_lb = np.where(scale > 0, lo * scale, hi * scale)
    exp_ub = np.where(scale > 0, hi * scale, lo * scale)
    np.testing.assert_allclose(r2["lb"][:, 20:], exp_lb, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r2["ub"][:, 20:], exp_ub, rtol=1e-12, atol=1e-13)


def test_brute_force_grid_tiny_net():
    w = wl.small_fc([2, 3, 3, 2], batch=1, eps=0.3, seed=51)
    r = orc.deeppoly(w.layers, w.centers, w.eps)
    L0, U0 = mat.box(w.centers, w.eps, 0.0, 1.0)
    g = np.linspace(0.0, 1.0, 1001)
    xx, yy = np.meshgrid(g, g, indexing="ij")
    x = np.stack([L0[0, 0] + (U0[0, 0] - L0[0, 0]) * xx.ravel(),
                  L0[0, 1] + (U0[0, 1] - L0[0, 1]) * yy.ravel()], axis=1)
    z = mat.forward_preactivations(w.layers, x)
    assert (z.min(axis=0) >= r["lb"][0] - 1e-12).all()
    assert (z.max(axis=0) <= r["ub"][0] + 1e-12).all()
    # layer 1 is an interval bound of a linear map: attained at a grid corner
    np.testing.assert_allclose(z.min(axis=0)[:3], r["lb"][0, :3], atol=1e-12)
    np.testing.assert_allclose(z.max(axis=0)[:3], r["ub"][0, :3], atol=1e-12)


def test_deeppoly_is_not_intersected_with_interval_bounds():
    """In the worked example the back-substituted lower bound of y1 (-7/8) is looser
    than the interval bound (-3/4): the listing takes l = backsubs_lower(...) alone."""
    g, layers = _w1()
    r = orc.deeppoly(layers, np.array([g["center"]], np.float32), g["eps"], *g["clip"])
    assert r["lb"][0, 2] == -0.875


def test_margins_flag_near_ties():
    g, layers = _w1(bias1=[0.0, 0.0])
    r = orc.deeppoly(layers, np.zeros((1, 2), np.float32), 1.0, -1.0, 1.0)
    assert r["margins"][0, 0] == 0.0
    g, layers = _w1()
    r = orc.deeppoly(layers, np.array([g["center"]], np.float32), g["eps"], *g["clip"])
    np.testing.assert_allclose(r["margins"][0, 0], 0.5 / 2.5)
