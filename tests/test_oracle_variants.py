"""Pins for the oracle's traversal-depth variants: DeepPoly_p (Section 6.2), and the IBP and
CROWN-IBP listings of Appendix C, which differ from DeepPoly only in how far each affine layer's
expressions are back-substituted before they are simplified against concrete bounds."""
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


def _w1():
    g = json.load(open(os.path.join(GOLD, "w1_example.json")))
    layers = [wl.Layer("fc", np.array(l["weight"], np.float32), np.array(l["bias"], np.float32),
                       relu_after=l["relu_after"]) for l in g["layers"]]
    return g, layers


def test_w1_hand_values_of_the_variants():
    g, layers = _w1()
    c = np.array([g["center"]], np.float32)
    v = g["variants"]
    runs = {"deeppoly_p1": orc.deeppoly(layers, c, g["eps"], *g["clip"], max_backsteps=1),
            "ibp": orc.ibp(layers, c, g["eps"], *g["clip"]),
            "crown_ibp": orc.crown_ibp(layers, c, g["eps"], *g["clip"])}
    for name, r in runs.items():
        np.testing.assert_allclose(r["lb"][0], _fr(v[name]["lb"]), rtol=0, atol=1e-14, err_msg=name)
        np.testing.assert_allclose(r["ub"][0], _fr(v[name]["ub"]), rtol=0, atol=1e-14, err_msg=name)
        if "codes" in v[name]:
            assert r["codes"][0].tolist() == v[name]["codes"], name


def _interval_propagation(layers, centers, eps, clip_lo, clip_hi):
    """Textbook interval arithmetic in centre/radius form (not the listing's sign-split form):
    mid' = A mid + b, rad' = |A| rad; ReLU applied to the end points."""
    L0, U0 = mat.box(centers, eps, clip_lo, clip_hi)
    lbs, ubs = [], []
    lo, up = L0, U0
    for layer in layers:
        A, b = mat.dense_matrix(layer), mat.dense_bias(layer)
        mid, rad = (lo + up) / 2, (up - lo) / 2
        m2, r2 = mid @ A.T + b, rad @ np.abs(A).T
        lbs.append(m2 - r2); ubs.append(m2 + r2)
        lo, up = (np.maximum(m2 - r2, 0), np.maximum(m2 + r2, 0)) if layer.relu_after else (m2 - r2, m2 + r2)
    return np.concatenate(lbs, axis=1), np.concatenate(ubs, axis=1)


NETS = [
    lambda: wl.small_fc([10, 24, 24, 24, 5], batch=3, eps=0.05, seed=21),
    lambda: wl.small_conv((2, 8, 8), [(4, 4, 2, 1), (6, 4, 2, 1)], [12, 4], batch=2, eps=0.03, seed=22),
    lambda: wl.make_config(0),
]


@pytest.mark.parametrize("make", NETS)
def test_ibp_is_interval_arithmetic(make):
    w = make()
    r = orc.ibp(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    lb, ub = _interval_propagation(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(r["lb"], lb, rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(r["ub"], ub, rtol=1e-11, atol=1e-11)
    r0 = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, max_backsteps=0)
    assert np.array_equal(r0["lb"], r["lb"]) and np.array_equal(r0["ub"], r["ub"])


@pytest.mark.parametrize("make", NETS)
def test_enough_steps_is_full_deeppoly(make):
    w = make()
    K = len(w.layers)
    full = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    for p in (K - 1, K, K + 5):
        r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, max_backsteps=p)
        assert np.array_equal(r["lb"], full["lb"]) and np.array_equal(r["ub"], full["ub"])
        assert np.array_equal(r["codes"], full["codes"])
    # per-layer counts: layer k needs k steps to reach the input
    r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=list(range(K)))
    assert np.array_equal(r["lb"], full["lb"]) and np.array_equal(r["ub"], full["ub"])
    # a uniform count and the same count per layer agree
    a = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, max_backsteps=1)
    b = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=[1] * K)
    assert np.array_equal(a["lb"], b["lb"]) and np.array_equal(a["ub"], b["ub"])


def _variants(K):
    return {"p0": [0] * K, "p1": [1] * K, "p2": [2] * K, "crown_ibp": [0] * (K - 1) + [-1],
            "mixed": [(-1 if k % 2 else 1) for k in range(K)]}


@pytest.mark.parametrize("make", NETS)
def test_matrix_form_agrees_on_the_variants(make):
    w = make()
    for name, steps in _variants(len(w.layers)).items():
        r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        lb, ub, codes = mat.deeppoly_matrix(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps=steps)
        np.testing.assert_allclose(r["lb"], lb, rtol=1e-10, atol=1e-10, err_msg=name)
        np.testing.assert_allclose(r["ub"], ub, rtol=1e-10, atol=1e-10, err_msg=name)
        assert np.array_equal(r["codes"], codes), name


def _samples(l0, u0, m, seed):
    n = l0.shape[0]
    u = wl.uniform01(seed, 78, m * n).reshape(m, n)
    x = l0 + (u0 - l0) * u
    x[m // 2:] = np.where(u[m // 2:] < 0.5, l0, u0)
    return x


@pytest.mark.parametrize("make", NETS[:2])
def test_variants_are_sound_on_samples(make):
    w = make()
    L0, U0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    for name, steps in _variants(len(w.layers)).items():
        r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        assert (r["lb"] <= r["ub"] + 1e-12).all(), name
        for b in range(w.batch):
            z = mat.forward_preactivations(w.layers, _samples(L0[b], U0[b], 50_000, seed=b))
            lb, ub = r["lb"][b], r["ub"][b]
            assert (z.min(axis=0) >= lb - 1e-9 * (1 + np.abs(lb))).all(), name
            assert (z.max(axis=0) <= ub + 1e-9 * (1 + np.abs(ub))).all(), name


def test_ibp_never_beats_crown_ibp_at_the_last_layer_on_a_linear_tail():
    """With every hidden neuron stable the last layer's back-substitution is exact, so CROWN-IBP's
    last-layer interval lies inside IBP's."""
    w = wl.small_fc([6, 10, 10, 3], batch=2, eps=0.0005, seed=33, b_sigma=5.0)
    a = orc.ibp(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    c = orc.crown_ibp(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    assert (c["codes"] <= 1).all()
    assert (c["lb"][:, -3:] >= a["lb"][:, -3:] - 1e-12).all()
    assert (c["ub"][:, -3:] <= a["ub"][:, -3:] + 1e-12).all()


# ---- SkipPoly listing (Appendix C): ReLU shapes expressed two layers back ----

def test_skippoly_w1_hand_values():
    """On the 2-2-2-1 example every slope the upper shapes multiply into the weights is a dyadic or a
    multiple of 1/19, and the hand evaluation of the SkipPoly listing gives DeepPoly's numbers: the shape of a
    ReLU neuron over the layer two back is its DeepPoly shape with the affine neuron's expression substituted."""
    g, layers = _w1()
    r = orc.skippoly(layers, np.array([g["center"]], np.float32), g["eps"], *g["clip"])
    np.testing.assert_allclose(r["lb"][0], _fr(g["lb"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(r["ub"][0], _fr(g["ub"]), rtol=0, atol=1e-14)
    assert r["codes"][0].tolist() == g["codes"]


@pytest.mark.parametrize("make", NETS)
def test_skippoly_has_deeppoly_precision(make):
    """Section 6.1: expressing the ReLU bounds two layers back does not change the bounds ("without
    sacrificing precision"); only the order of the floating-point products differs."""
    w = make()
    a = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    b = orc.skippoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(b["lb"], a["lb"], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(b["ub"], a["ub"], rtol=1e-11, atol=1e-11)
    assert np.array_equal(a["codes"], b["codes"])


def test_skippoly_soundness_and_missing_relu():
    w = wl.small_fc([8, 16, 16, 16, 4], batch=2, eps=0.1, seed=35)
    w.layers[1].relu_after = False            # an affine layer directly on an affine layer
    r = orc.skippoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    a = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(r["lb"], a["lb"], rtol=1e-11, atol=1e-11)
    L0, U0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    for b in range(w.batch):
        z = mat.forward_preactivations(w.layers, _samples(L0[b], U0[b], 50_000, seed=b))
        assert (z.min(axis=0) >= r["lb"][b] - 1e-9 * (1 + np.abs(r["lb"][b]))).all()
        assert (z.max(axis=0) <= r["ub"][b] + 1e-9 * (1 + np.abs(r["ub"][b]))).all()


# ---- ReuseCert listing (Appendix C): shapes kept over the input layer and reused ----

def test_reusecert_w1_hand_values():
    g, layers = _w1()
    v = g["variants"]["reusecert"]
    r = orc.reusecert(layers, np.array([g["center"]], np.float32), g["eps"], *g["clip"])
    np.testing.assert_allclose(r["lb"][0], _fr(v["lb"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(r["ub"][0], _fr(v["ub"]), rtol=0, atol=1e-14)
    assert r["codes"][0].tolist() == v["codes"]


@pytest.mark.parametrize("make", NETS)
def test_reusecert_matrix_form_agrees(make):
    w = make()
    r = orc.reusecert(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    lb, ub, codes = mat.reusecert_matrix(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(r["lb"], lb, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(r["ub"], ub, rtol=1e-10, atol=1e-10)
    assert np.array_equal(r["codes"], codes)


def test_reusecert_equals_deeppoly_up_to_the_second_affine_layer_and_when_stable():
    """One traversal round is all DeepPoly does at the second affine layer, so the first two layers agree;
    with every neuron stable both are the exact range of the linear map."""
    w = wl.small_fc([10, 24, 24, 24, 5], batch=3, eps=0.05, seed=21)
    a = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    r = orc.reusecert(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    np.testing.assert_allclose(r["lb"][:, :48], a["lb"][:, :48], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(r["ub"][:, :48], a["ub"][:, :48], rtol=1e-12, atol=1e-12)
    assert not np.allclose(r["lb"][:, 48:], a["lb"][:, 48:], rtol=1e-6, atol=1e-6)   # later layers differ
    s = wl.small_fc([6, 10, 10, 10, 3], batch=2, eps=0.0005, seed=33, b_sigma=5.0)
    a = orc.deeppoly(s.layers, s.centers, s.eps, s.clip_lo, s.clip_hi)
    r = orc.reusecert(s.layers, s.centers, s.eps, s.clip_lo, s.clip_hi)
    assert (a["codes"] <= 1).all()
    np.testing.assert_allclose(r["lb"], a["lb"], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(r["ub"], a["ub"], rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("make", NETS[:2])
def test_reusecert_is_sound_on_samples(make):
    w = make()
    r = orc.reusecert(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    L0, U0 = mat.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
    assert (r["lb"] <= r["ub"] + 1e-12).all()
    for b in range(w.batch):
        z = mat.forward_preactivations(w.layers, _samples(L0[b], U0[b], 50_000, seed=b))
        assert (z.min(axis=0) >= r["lb"][b] - 1e-9 * (1 + np.abs(r["lb"][b]))).all()
        assert (z.max(axis=0) <= r["ub"][b] + 1e-9 * (1 + np.abs(r["ub"][b]))).all()
