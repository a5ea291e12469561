"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle,
element by element, on the same seeded inputs."""
import numpy as np
import pytest

from oracle import deeppoly_oracle as orc
from paper_2507_20055_b200 import workloads as wl
from parity_util import cached_oracle, compare, run_gpu

pytestmark = pytest.mark.gpu


def _oracle(w, boxes=None):
    c = w.centers if boxes is None else w.centers[np.asarray(boxes)]
    return orc.deeppoly(w.layers, c, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)


MODES = {"ffma": 1, "tc": 2}


@pytest.mark.parametrize("mode", ["ffma", "tc"])
@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config_full_batch(idx, mode):
    w = wl.make_config(idx)
    g = run_gpu(w, contraction=MODES[mode])
    assert g["paths"] & MODES[mode] or idx == 3
    compare(g, _oracle(w), label=f"{w.name}/{mode}")


@pytest.mark.parametrize("mode", ["ffma", "tc", "tc16", "auto"])
def test_config5_all_boxes(mode):
    """784 -> 1024 x 6 -> 10, 128 boxes, the benchmark's launch configuration: every box against the oracle
    (one oracle run of a few minutes on the host cores, shared by the modes and kept on disk).  A box with a
    near-tie neuron is compared up to the layer where the tie is resolved differently, not dropped."""
    w = wl.make_config(4)
    g = run_gpu(w, contraction={"ffma": 1, "tc": 2, "tc16": 3, "auto": 0}[mode])
    if mode in ("tc16", "auto"):
        assert g["paths"] & 16            # AUTO proves the fp16 range of the wide layers' traversals at create
    r = compare(g, cached_oracle(w), label=f"{w.name}/{mode}", min_compared=0.9)
    assert r["boxes"] == 128


SMALL = {
    "ragged_widths": lambda: wl.small_fc([37, 50, 33, 70, 10], batch=5, eps=0.03, seed=61),
    "one_hidden": lambda: wl.small_fc([20, 45, 7], batch=3, eps=0.1, seed=62),
    "single_layer": lambda: wl.small_fc([30, 12], batch=4, eps=0.1, seed=63),
    "wide_then_narrow": lambda: wl.small_fc([64, 300, 130, 257, 3], batch=9, eps=0.02, seed=64),
    "relu_on_last": lambda: wl.small_fc([16, 40, 40, 8], batch=2, eps=0.05, seed=65, relu_last=True),
    "conv_small": lambda: wl.small_conv((2, 9, 7), [(5, 3, 2, 1), (6, 3, 1, 1)], [20, 4], batch=3, eps=0.02, seed=66),
    "conv_k4s2": lambda: wl.small_conv((3, 12, 12), [(8, 4, 2, 1), (12, 4, 2, 1)], [30, 5], batch=4, eps=0.01, seed=67),
    "conv_only_then_fc": lambda: wl.small_conv((1, 10, 10), [(20, 5, 1, 0)], [6], batch=2, eps=0.05, seed=68),
    "conv_stride3": lambda: wl.small_conv((2, 11, 13), [(4, 3, 3, 2)], [9, 3], batch=2, eps=0.05, seed=69),
}


@pytest.mark.parametrize("mode", ["ffma", "tc"])
@pytest.mark.parametrize("name", sorted(SMALL))
def test_small_and_ragged(name, mode):
    w = SMALL[name]()
    if mode == "tc" and len(w.layers) < 2:
        pytest.skip("a single layer has no back-step")
    compare(run_gpu(w, contraction=MODES[mode]), _oracle(w), label=f"{name}/{mode}")


def test_missing_relu_in_the_middle():
    w = wl.small_fc([24, 40, 36, 40, 6], batch=3, eps=0.05, seed=71)
    w.layers[1].relu_after = False
    compare(run_gpu(w), _oracle(w), label="no_relu_mid")


def test_eps_zero_degenerate_box():
    w = wl.small_fc([24, 40, 40, 6], batch=3, eps=0.0, seed=72)
    g, r = run_gpu(w), _oracle(w)
    assert set(np.unique(g["codes"])) <= {0, 1}
    np.testing.assert_allclose(g["lb"], g["ub"], rtol=0, atol=1e-5)
    compare(g, r, label="eps0")


def test_no_clipping_and_large_eps():
    w = wl.small_fc([12, 30, 30, 5], batch=2, eps=0.7, seed=73, clip=(-float("inf"), float("inf")))
    compare(run_gpu(w), _oracle(w), label="noclip")


def test_batch_smaller_than_max_batch_and_reuse():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([33, 64, 64, 10], batch=6, eps=0.04, seed=74)
    r = _oracle(w)
    net = binding.CertNet(w.layers, 16)
    try:
        c = torch.from_numpy(w.centers).cuda()
        for batch in (6, 2, 6):          # the workspace is reused across calls
            lb, ub = net.deeppoly_bounds(c[:batch].contiguous(), w.eps)
            torch.cuda.synchronize()
            g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(),
                 "codes": net.branch_codes(batch).cpu().numpy(), "status": net.last_status(), "layers": w.layers}
            sub = {k: v[:batch] for k, v in r.items()}
            compare(g, sub, label=f"reuse_b{batch}")
    finally:
        net.destroy()


def test_host_buffer_entry_point():
    w = wl.small_fc([33, 64, 64, 10], batch=4, eps=0.04, seed=75)
    compare(run_gpu(w, host_api=True), _oracle(w), label="host_api")


def test_non_default_stream():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([33, 64, 64, 10], batch=4, eps=0.04, seed=76)
    r = _oracle(w)
    net = binding.CertNet(w.layers, w.batch)
    try:
        s = torch.cuda.Stream()
        c = torch.from_numpy(w.centers).cuda()
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            lb, ub = net.deeppoly_bounds(c, w.eps, stream=s)
            codes = net.branch_codes(w.batch, stream=s)
        s.synchronize()
        g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": codes.cpu().numpy(),
             "status": net.last_status(s.cuda_stream), "layers": w.layers}
        compare(g, r, label="stream")
    finally:
        net.destroy()


def test_error_codes_on_device():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([8, 8, 4], batch=2, eps=0.1, seed=77)
    net = binding.CertNet(w.layers, 2)
    try:
        c = torch.zeros((3, 8), device="cuda")
        out = torch.empty((3, net.n_total), device="cuda")
        L = binding.lib
        assert L.cert_deeppoly_bounds(net._h, c.data_ptr(), 0.1, 3, out.data_ptr(), out.data_ptr(), None) == 4
        assert L.cert_deeppoly_bounds(net._h, None, 0.1, 1, out.data_ptr(), out.data_ptr(), None) == 1
        assert L.cert_deeppoly_bounds(net._h, c.data_ptr(), -1.0, 1, out.data_ptr(), out.data_ptr(), None) == 1
        assert L.cert_deeppoly_bounds(net._h, c.data_ptr(), float("nan"), 1, out.data_ptr(), out.data_ptr(), None) == 1
        assert L.cert_deeppoly_bounds(net._h, c.data_ptr(), 0.1, 0, out.data_ptr(), out.data_ptr(), None) == 1
    finally:
        net.destroy()


# ---- bounded traversals: DeepPoly_p (Section 6.2), IBP and CROWN-IBP listings (Appendix C) ----

VARIANT_NETS = {
    "fc_ragged": lambda: wl.small_fc([37, 50, 33, 70, 40, 10], batch=5, eps=0.03, seed=81),
    "fc_wide": lambda: wl.small_fc([64, 300, 130, 257, 3], batch=6, eps=0.02, seed=82),
    "conv": lambda: wl.small_conv((3, 12, 12), [(8, 4, 2, 1), (12, 4, 2, 1)], [30, 5], batch=4, eps=0.01, seed=83),
    "fc6x100": lambda: wl.make_config(1, batch=8),
}


def _variant_steps(K):
    return {"ibp": [0] * K, "p1": [1] * K, "p2": [2] * K, "crown_ibp": [0] * (K - 1) + [-1],
            "mixed": [(-1 if k % 2 else 1) for k in range(K)], "full_as_counts": list(range(K))}


@pytest.mark.parametrize("mode", ["ffma", "tc"])
@pytest.mark.parametrize("name", sorted(VARIANT_NETS))
def test_bounded_traversals(name, mode):
    w = VARIANT_NETS[name]()
    for vname, steps in _variant_steps(len(w.layers)).items():
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        g = run_gpu(w, contraction=MODES[mode], backsteps=steps)
        compare(g, ref, label=f"{name}/{vname}/{mode}")


def test_bounded_traversal_wrappers_and_null_array():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([20, 32, 32, 32, 6], batch=3, eps=0.05, seed=84)
    net = binding.CertNet(w.layers, w.batch)
    try:
        c = torch.from_numpy(w.centers).cuda()
        runs = {"ibp": (net.ibp_bounds(c, w.eps), orc.ibp(w.layers, w.centers, w.eps)),
                "crown_ibp": (net.crown_ibp_bounds(c, w.eps), orc.crown_ibp(w.layers, w.centers, w.eps)),
                "p1": (net.deeppoly_p_bounds(c, w.eps, 1), orc.deeppoly(w.layers, w.centers, w.eps, max_backsteps=1)),
                "null": (net.backsub_bounds(c, w.eps, None), orc.deeppoly(w.layers, w.centers, w.eps))}
        for name, ((lb, ub), ref) in runs.items():
            torch.cuda.synchronize()
            g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": ref["codes"], "status": net.last_status(), "layers": w.layers}
            compare(g, ref, label=name)
    finally:
        net.destroy()


@pytest.mark.parametrize("name", ["fc_ragged", "conv"])
def test_fused_steps_against_the_skippoly_listing(name):
    """The GPU path takes a ReLU layer and the affine layer below it in one kernel, which is the traversal
    of the SkipPoly listing (Appendix C: ReLU shapes expressed two layers back, one round per ReLU layer)."""
    w = VARIANT_NETS[name]()
    ref = orc.skippoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    compare(run_gpu(w), ref, label=f"{name}/skippoly")


# ---- conv-sourced rows as dense maps and as receptive-field patches ----

CONV_NETS = {
    "convsmall": lambda: wl.make_config(3, batch=4),
    "k3s2_k3s1": lambda: wl.small_conv((2, 9, 7), [(5, 3, 2, 1), (6, 3, 1, 1)], [20, 4], batch=3, eps=0.02, seed=66),
    "k4s2_k4s2": lambda: wl.small_conv((3, 12, 12), [(8, 4, 2, 1), (12, 4, 2, 1)], [30, 5], batch=4, eps=0.01, seed=67),
    "three_convs": lambda: wl.small_conv((2, 20, 18), [(4, 3, 1, 1), (6, 4, 2, 1), (8, 3, 2, 0)], [12, 3], batch=2,
                                         eps=0.01, seed=85),
    "k5s1p0_k2s2": lambda: wl.small_conv((1, 14, 14), [(6, 5, 1, 0), (4, 2, 2, 0)], [5], batch=2, eps=0.03, seed=86),
    # map rows (channels x width) that are multiples of 32 floats: the dense steps take the banded tensor-core form
    "pow2_two_convs": lambda: wl.small_conv((2, 32, 32), [(4, 4, 2, 1), (8, 4, 2, 1)], [12, 4], batch=2, eps=0.01, seed=89),
    "pow2_first_only": lambda: wl.small_conv((2, 16, 16), [(8, 4, 2, 1), (6, 4, 2, 1)], [20, 5], batch=3, eps=0.01, seed=90),
    "pow2_k3s1": lambda: wl.small_conv((4, 8, 8), [(8, 3, 1, 1), (8, 3, 1, 1)], [10, 3], batch=2, eps=0.01, seed=95),
}


@pytest.mark.parametrize("form", ["dense", "patches_fma", "patches_tc"])
@pytest.mark.parametrize("name", sorted(CONV_NETS))
def test_conv_rows_dense_and_patches(name, form):
    """Rows of a conv layer over conv layers: as dense maps, as receptive-field patches on the FMA units (one
    warp per row), and as patches on the tensor cores (the conv layer as a dense window-to-window matrix)."""
    w = CONV_NETS[name]()
    ref = _oracle(w)
    patches = form != "dense"
    contraction = MODES["ffma"] if form == "patches_fma" else None
    g = run_gpu(w, conv_patches=patches, contraction=contraction)
    # the small nets' windows are not much smaller than their maps: those stay dense either way
    expect_patches = patches and name in ("convsmall", "three_convs", "k5s1p0_k2s2")
    if not name.startswith("pow2"):
        assert bool(g["paths"] & 8) == expect_patches
    if expect_patches and form == "patches_tc":
        assert g["paths"] & 2
    banded = form != "patches_fma" and name in ("convsmall", "pow2_two_convs", "pow2_first_only", "pow2_k3s1")
    assert bool(g["paths"] & 64) == banded
    compare(g, ref, label=f"{name}/{form}")
    steps = [0] + [1] * (len(w.layers) - 1)
    ref1 = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
    compare(run_gpu(w, conv_patches=patches, contraction=contraction, backsteps=steps), ref1, label=f"{name}/{form}/p1")


def test_banded_conv_steps_ragged_batch_and_traversal_depths():
    """Dense maps band by band on the tensor cores: fewer boxes than the net was made for, rows that do not fill the
    last 256-row panel, traversals that stop on a conv layer's input map, and the FMA kernels as cross-check."""
    w = wl.small_conv((2, 32, 32), [(4, 4, 2, 1), (8, 4, 2, 1)], [12, 4], batch=3, eps=0.01, seed=96)
    K = len(w.layers)
    for vname, steps in {"full": None, "p1": [1] * K, "p2": [2] * K, "crown_ibp": [0] * (K - 1) + [-1],
                         "mixed": [0, 1, -1, 2]}.items():
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        g = run_gpu(w, max_batch=w.batch + 2, backsteps=steps, conv_patches=False)
        if vname in ("full", "p2", "crown_ibp"):
            assert g["paths"] & 64, vname
        compare(g, ref, label=f"banded/{vname}")
        compare(run_gpu(w, max_batch=w.batch + 2, backsteps=steps, conv_patches=False, contraction=MODES["ffma"]), ref,
                label=f"banded/{vname}/ffma cross-check")


def test_conv_patches_on_tensor_cores_ragged_batch():
    """Fewer boxes than the net was made for, rows not a multiple of the 256-row panel."""
    w = wl.small_conv((2, 20, 18), [(4, 3, 1, 1), (6, 4, 2, 1), (8, 3, 2, 0)], [12, 3], batch=3, eps=0.01, seed=87)
    ref = _oracle(w)
    g = run_gpu(w, max_batch=5, conv_patches=True)
    assert g["paths"] & 8 and g["paths"] & 2
    compare(g, ref, label="three_convs/ragged")


# ---- ReuseCert (Appendix C listing): shapes kept over the input layer ----

REUSE_NETS = {
    "fc_ragged": lambda: wl.small_fc([37, 50, 33, 70, 40, 10], batch=5, eps=0.03, seed=81),
    "fc_wide": lambda: wl.small_fc([64, 300, 130, 257, 3], batch=6, eps=0.02, seed=82),
    "n0_multiple_of_32": lambda: wl.small_fc([64, 96, 96, 8], batch=3, eps=0.02, seed=87),
    "fc6x100": lambda: wl.make_config(1, batch=8),
    "fc3x50": lambda: wl.make_config(0),
}


# ReuseCert feeds every layer with the rounded shapes of the layer below, so float32 rounding compounds through
# the layers where DeepPoly restarts each traversal from the exact weights.  The library serves it in the fp16
# split only, which holds the common tolerance.
REUSE_TOL = 1e-4


def _run_reusecert(w, max_batch=None, contraction=None):
    import torch
    from paper_2507_20055_b200 import binding
    net = binding.CertNet(w.layers, max_batch or w.batch, w.clip_lo, w.clip_hi)
    try:
        if contraction is not None:
            net.set_contraction(contraction)
        net.enable_reusecert()
        c = torch.from_numpy(np.ascontiguousarray(w.centers)).cuda()
        out = []
        for _ in range(2):                      # the second call reuses every buffer
            lb, ub = net.reusecert_bounds(c, w.eps)
            torch.cuda.synchronize()
            out.append({"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(),
                        "codes": net.branch_codes(w.batch).cpu().numpy(), "status": net.last_status(), "layers": w.layers})
        # DeepPoly on the same net still works after ReuseCert was enabled
        lb, ub = net.deeppoly_bounds(c, w.eps)
        torch.cuda.synchronize()
        dp = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": net.branch_codes(w.batch).cpu().numpy(),
              "status": net.last_status(), "layers": w.layers}
    finally:
        net.destroy()
    return out, dp


@pytest.mark.parametrize("mode", ["auto", "tc16"])
@pytest.mark.parametrize("name", sorted(REUSE_NETS))
def test_reusecert(name, mode):
    w = REUSE_NETS[name]()
    ref = orc.reusecert(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    out, dp = _run_reusecert(w, max_batch=w.batch + 3, contraction={"auto": 0, "tc16": 3}[mode])
    for i, g in enumerate(out):
        compare(g, ref, label=f"reusecert/{name}/{mode}/call{i}", tol=REUSE_TOL)
    assert np.array_equal(out[0]["lb"], out[1]["lb"]) and np.array_equal(out[0]["ub"], out[1]["ub"])
    compare(dp, _oracle(w), label=f"deeppoly_after_reusecert/{name}")


def test_reusecert_needs_enable_and_fc_layers():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([8, 8, 4], batch=2, eps=0.1, seed=77)
    net = binding.CertNet(w.layers, 2)
    try:
        c = torch.from_numpy(w.centers).cuda()
        out = torch.empty((2, net.n_total), device="cuda")
        assert binding.lib.cert_reusecert_bounds(net._h, c.data_ptr(), 0.1, 2, out.data_ptr(), out.data_ptr(), None) == 2
    finally:
        net.destroy()
    wc = wl.small_conv((1, 10, 10), [(20, 5, 1, 0)], [6], batch=2, eps=0.05, seed=68)
    net = binding.CertNet(wc.layers, 2)
    try:
        assert binding.lib.cert_net_enable_reusecert(net._h) == 2
    finally:
        net.destroy()
    # a net pinned to the TF32 split or the FMA units is refused: ReuseCert runs in the fp16 split only
    net = binding.CertNet(w.layers, 2)
    try:
        net.enable_reusecert()
        c = torch.from_numpy(w.centers).cuda()
        out = torch.empty((2, net.n_total), device="cuda")
        for mode in (1, 2):
            net.set_contraction(mode)
            assert binding.lib.cert_reusecert_bounds(net._h, c.data_ptr(), 0.1, 2, out.data_ptr(), out.data_ptr(), None) == 2
    finally:
        net.destroy()


@pytest.mark.parametrize("mode", ["auto"])
def test_reusecert_config5_all_boxes(mode):
    """784 -> 1024 x 6 -> 10, 128 boxes on the GPU (the benchmark's launch configuration), every box against the
    oracle.  With 6144 ReLU neurons per box and ReuseCert's wider bounds most boxes have some neuron whose sign
    test is within float32 noise of zero; such a box is compared up to the layer where the GPU resolves a
    near-tie differently."""
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.make_config(4)
    ref = cached_oracle(w, "reusecert")
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        net.set_contraction({"auto": 0, "tc16": 3}[mode])
        net.enable_reusecert()
        lb, ub = net.reusecert_bounds(torch.from_numpy(w.centers).cuda(), w.eps)
        torch.cuda.synchronize()
        g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": net.branch_codes(w.batch).cpu().numpy(),
             "status": net.last_status(), "layers": w.layers}
    finally:
        net.destroy()
    compare(g, ref, label=f"reusecert/fc6x1024/{mode}", tol=REUSE_TOL, min_compared=0.8)


# ---- fp16-split tensor-core contraction (CERT_CONTRACTION_TC3XFP16), nets of FC layers ----

TC16 = 3
FC_NETS = {
    "fc3x50": lambda: wl.make_config(0),
    "fc6x100": lambda: wl.make_config(1),
    "fc9x200": lambda: wl.make_config(2),
    "ragged_widths": SMALL["ragged_widths"],
    "one_hidden": SMALL["one_hidden"],
    "wide_then_narrow": SMALL["wide_then_narrow"],
    "relu_on_last": SMALL["relu_on_last"],
    "fc_ragged5": VARIANT_NETS["fc_ragged"],
}


@pytest.mark.parametrize("chain", [True, False])
@pytest.mark.parametrize("name", sorted(FC_NETS))
def test_fp16_split_contraction(name, chain, monkeypatch):
    """Narrow nets: a whole traversal per launch (the coefficient panel stays in shared memory), and, with
    CERT_CHAIN=0 at create, one launch per back-step as for wide nets."""
    if not chain:
        monkeypatch.setenv("CERT_CHAIN", "0")
    w = FC_NETS[name]()
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 16
    narrow = max(l.weight.shape[0] for l in w.layers[:-1]) <= 256
    assert bool(g["paths"] & 32) == (chain and narrow)
    compare(g, _oracle(w), label=f"{name}/tc16/chain={chain}")


@pytest.mark.parametrize("name", sorted(FC_NETS))
def test_fp16_split_two_pass_form(name, monkeypatch):
    """One launch per back-step with CERT_TC16_ONE_PASS=0 at create: the pair keeps its lo part times 2^11 and a
    k-block is staged twice (the form ReuseCert's contraction always runs).  The default, one pass over K with both
    operands times a power of two, is what every other fp16-split test of the per-step kernel runs."""
    monkeypatch.setenv("CERT_CHAIN", "0")
    monkeypatch.setenv("CERT_TC16_ONE_PASS", "0")
    w = FC_NETS[name]()
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 16 and not g["paths"] & 32
    compare(g, _oracle(w), label=f"{name}/tc16/two passes")


def test_fp16_split_one_pass_scale_follows_the_proved_bound(monkeypatch):
    """Coefficients of the one-pass form travel times 2^a, a = what the layer's proved bound leaves of the fp16 range
    (at most 14).  Weights of +-1.5 on 40-wide layers make the bound grow sixtyfold per layer, so a falls from 14 to 3
    along the net and the output layer, without a proof, runs at a = 0 when the mode is forced: every layer must
    agree with the oracle, and none may raise the range flag (run_gpu checks the status word)."""
    from paper_2507_20055_b200 import binding
    monkeypatch.setenv("CERT_CHAIN", "0")
    w = wl.small_fc([64, 40, 40, 40, 40, 6], batch=5, eps=0.002, seed=97)
    for l in w.layers[1:]:
        l.weight[...] = np.where(l.weight >= 0, 1.5, -1.5).astype(np.float32)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        bounds = [net.fp16_coefficient_bound(k) for k in range(1, len(w.layers))]
    finally:
        net.destroy()
    assert bounds[0] <= 60000.0 / 16384                     # a = 14
    assert 60000.0 / 16 < bounds[2] <= 60000.0              # 0 <= a <= 3
    assert bounds[3] > 60000.0                              # no proof
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 16 and not g["paths"] & 32
    compare(g, _oracle(w), min_good_fraction=0.4, label="pm1.5/tc16 one pass")
    g = run_gpu(w)                                          # AUTO: the output layer on trial at a = 4
    assert g["paths"] & 128
    compare(g, _oracle(w), min_good_fraction=0.4, label="pm1.5/auto")


@pytest.mark.parametrize("sizes", [[784, 600, 330, 7], [600, 544, 700, 258, 3], [1000, 288, 513, 10]])
@pytest.mark.parametrize("mode", ["tc16", "tc16_two_pass", "auto"])
def test_fp16_split_unequal_column_tiles(sizes, mode, monkeypatch):
    """Layers wider than 256 (one launch per back-step) whose widths make the column tiles of a row panel unequal
    (600 = 224 + 192 + 192, 784 = 224 + 3 x 192, 330 -> 192 + 160), ragged K blocks and row panels that the
    2 x batch x n_k rows do not fill."""
    if mode == "tc16_two_pass":
        monkeypatch.setenv("CERT_TC16_ONE_PASS", "0")
    w = wl.small_fc(sizes, batch=3, eps=0.005, seed=sum(sizes))
    g = run_gpu(w, contraction=0 if mode == "auto" else TC16, max_batch=4)
    assert g["paths"] & 16 and not g["paths"] & 32
    compare(g, _oracle(w), min_good_fraction=0.6, label=f"{sizes}/{mode}")


@pytest.mark.parametrize("mode", ["tc16", "auto"])
def test_fp16_split_unequal_column_tiles_with_residual_connections(mode):
    """272-wide layers (column tiles of 160 and 128) in a net with residual connections: the joining epilogue reads the
    waiting pair at the narrower tile's columns."""
    w = wl.residual_fc(300, 272, 2, 6, batch=3, eps=0.01, seed=41)
    g = run_gpu(w, contraction=0 if mode == "auto" else TC16, max_batch=4)
    assert g["paths"] & 16
    compare(g, _oracle(w), min_good_fraction=0.6, label=f"residual 272-wide/{mode}")


@pytest.mark.parametrize("batch", [1, 3])
def test_fc6x1024_small_batches_take_more_column_tiles(batch):
    """784 -> 1024 x 6 -> 10 on one and three boxes: 8 and 24 row panels per contraction, too few to give each of the
    74 CTA pairs a 256-column tile, so the launches take as many narrower column tiles as keep them
    one wave (the output layer's traversal sixteen); every box against the oracle."""
    w = wl.make_config(4, batch=batch + 1)
    w.centers = np.ascontiguousarray(w.centers[1:])          # (the first box has a near-tie neuron)
    g = run_gpu(w, max_batch=batch + 1)
    assert g["paths"] & 16
    compare(g, _oracle(w), label=f"fc6x1024/{batch} boxes")


def test_fp16_split_chain_wide_input_and_many_layers():
    """A CIFAR-sized input (14 column tiles in the concretising step) and the deepest net the chain kernel's
    parameter block takes (12 layers); one layer more goes back to one launch per back-step."""
    w = wl.small_fc([3072, 100, 100, 100, 10], batch=3, eps=0.004, seed=92)
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 32
    compare(g, _oracle(w), label="cifar_input/tc16 chain")
    w = wl.small_fc([30] + [40] * 11 + [5], batch=2, eps=0.002, seed=93)          # 12 affine layers
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 32
    compare(g, _oracle(w), min_good_fraction=0.4, label="12 layers/tc16 chain")
    w = wl.small_fc([30] + [40] * 12 + [5], batch=2, eps=0.002, seed=94)          # 13 affine layers
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 16 and not g["paths"] & 32
    compare(g, _oracle(w), min_good_fraction=0.4, label="13 layers/tc16 per step")


def test_fp16_split_chain_bounded_traversals_ragged_batch_and_missing_relu():
    w = VARIANT_NETS["fc_ragged"]()
    for vname, steps in _variant_steps(len(w.layers)).items():
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        g = run_gpu(w, contraction=TC16, backsteps=steps, max_batch=w.batch + 2)
        compare(g, ref, label=f"fc_ragged/{vname}/tc16 chain")
    w = wl.small_fc([24, 40, 36, 40, 6], batch=3, eps=0.05, seed=71)
    w.layers[1].relu_after = False
    g = run_gpu(w, contraction=TC16)
    assert g["paths"] & 32
    compare(g, _oracle(w), label="no_relu_mid/tc16 chain")


def test_fp16_split_bounded_traversals_and_missing_relu():
    w = VARIANT_NETS["fc_wide"]()
    for vname, steps in _variant_steps(len(w.layers)).items():
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, backsteps_per_layer=steps)
        compare(run_gpu(w, contraction=TC16, backsteps=steps), ref, label=f"fc_wide/{vname}/tc16")
    w = wl.small_fc([24, 40, 36, 40, 6], batch=3, eps=0.05, seed=71)
    w.layers[1].relu_after = False
    compare(run_gpu(w, contraction=TC16), _oracle(w), label="no_relu_mid/tc16")


def test_fp16_split_is_refused_for_conv_nets_and_flags_its_range():
    import torch
    from paper_2507_20055_b200 import binding
    wc = wl.small_conv((1, 10, 10), [(20, 5, 1, 0)], [6], batch=2, eps=0.05, seed=68)
    net = binding.CertNet(wc.layers, 2)
    try:
        assert binding.lib.cert_net_set_contraction(net._h, TC16) == 2      # CERT_ERR_UNSUPPORTED
    finally:
        net.destroy()
    # weights of 300 make second-layer coefficients of 9e4 > 65504: the range flag must come up
    w = _pm300_net()
    net = binding.CertNet(w.layers, 2, -1e30, 1e30)
    try:
        net.set_contraction(TC16)
        net.deeppoly_bounds(torch.from_numpy(w.centers).cuda(), w.eps)
        torch.cuda.synchronize()
        assert net.last_status() == 7                                          # CERT_ERR_RANGE
        assert net.last_status() == 0                                          # the flag is cleared by the read
    finally:
        net.destroy()


def _pm300_net():
    w = wl.small_fc([8, 16, 16, 4], batch=2, eps=0.01, seed=88, clip=(-1e30, 1e30))
    for l in w.layers:
        l.weight = (np.sign(l.weight) * 300.0).astype(np.float32)
    return w


def test_auto_takes_the_fp16_split_only_where_the_weights_prove_its_range():
    """CERT_CONTRACTION_AUTO, decided per layer: the largest entry of |W_k| ... |W_j| bounds every coefficient the
    traversal of layer k can hold.  Weights of +-300 in a 8-16-16-4 net: the traversal of layer 1 holds |W_1| = 300
    (fp16 split), that of layer 2 could reach 16 * 300 * 300 > 65504 and must run in the TF32 split; the bounds
    are the oracle's.  An ordinary net passes the proof everywhere."""
    from paper_2507_20055_b200 import binding
    w = _pm300_net()
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        assert net.fp16_coefficient_bound(1) == 300.0
        assert net.fp16_coefficient_bound(2) >= 16 * 300.0 * 300.0 * 0.999
        assert net.fp16_coefficient_bound() == net.fp16_coefficient_bound(2)
        assert net.fp16_coefficient_bound(3) == -1.0            # no such layer
    finally:
        net.destroy()
    g = run_gpu(w)
    # layer 2 runs in the fp16 split on trial, overflows, and its TF32 re-run takes over (bit 7: a re-run was enqueued)
    assert g["paths"] & 2 and g["paths"] & 16 and g["paths"] & 128
    compare(g, _oracle(w), label="pm300/auto")
    w = wl.small_fc([33, 64, 300, 64, 10], batch=4, eps=0.04, seed=75)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        assert net.auto_contraction() == 3
        # the bounds really are the largest entries of the products of the absolute weights
        a = [np.abs(l.weight.astype(np.float64)) for l in w.layers]
        expect = {1: a[1].max(), 2: max(a[2].max(), (a[2] @ a[1]).max()),
                  3: max(a[3].max(), (a[3] @ a[2]).max(), (a[3] @ a[2] @ a[1]).max())}
        for k, e in expect.items():
            assert abs(net.fp16_coefficient_bound(k) - e) <= 1e-5 * e
    finally:
        net.destroy()
    g = run_gpu(w)
    assert g["paths"] & 16 and not g["paths"] & 1
    compare(g, _oracle(w), label="ordinary/auto")


def test_auto_runs_unproven_layers_in_the_fp16_split_on_trial():
    """784 -> 200 x 9 -> 10: the products of the absolute weights pass 60000 from the eighth layer on although the
    real coefficients stay small.  AUTO runs those layers in the fp16 split all the same, each on a status word of
    its own, and enqueues the same traversal in the TF32 split with kernels that do nothing unless that word came
    up.  Here it does not: the bounds are the fp16 split's, and the call's own status stays clean."""
    from paper_2507_20055_b200 import binding
    w = wl.make_config(2, batch=6)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        unproven = [k for k in range(1, len(w.layers)) if net.fp16_coefficient_bound(k) > 60000.0]
        assert unproven and min(unproven) >= 5
    finally:
        net.destroy()
    ref = _oracle(w)
    g = run_gpu(w)
    assert g["paths"] & 32 and g["paths"] & 128 and not g["paths"] & 1
    compare(g, ref, label="fc9x200/auto on trial")
    # forced, the layers without a proof keep the whole fp16 range (coefficients times 1 instead of times 16): the
    # same bounds up to the rounding of the smallest lo parts
    forced = run_gpu(w, contraction=TC16)
    compare(forced, ref, label="fc9x200/fp16 split forced")
    for key in ("lb", "ub"):
        assert np.all(np.abs(forced[key] - g[key]) <= 2e-6 * (1.0 + np.abs(g[key])))
    # ... and not the TF32 split's: the re-run behind the trial did nothing
    tf32 = run_gpu(w, contraction=2)
    last = slice(-w.layers[-1].weight.shape[0], None)
    assert not np.array_equal(tf32["lb"][:, last], g["lb"][:, last])


def test_host_calls_report_the_device_status():
    """The host-buffer calls wait for their results, so they also read the status word: an fp16 overflow or a
    run-out wait comes back as an error code, never as bounds with CERT_OK."""
    from paper_2507_20055_b200 import binding
    w = _pm300_net()
    ref = _oracle(w)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        net.set_contraction(TC16)                       # forced: the coefficients leave the fp16 range
        with pytest.raises(binding.CertError) as e:
            net.deeppoly_bounds_host(w.centers, w.eps)
        assert e.value.code == 7                        # CERT_ERR_RANGE
        assert net.last_status() == 0                   # the host call cleared the word
        net.set_contraction(0)
        lb, ub = net.deeppoly_bounds_host(w.centers, w.eps)
        g = {"lb": lb, "ub": ub, "codes": net.branch_codes(w.batch).cpu().numpy(), "status": net.last_status(),
             "layers": w.layers}
        compare(g, ref, label="pm300/host/auto")
        net.selftest_bounded_wait()                     # raises the time-out bit on the same stream
        with pytest.raises(binding.CertError) as e:
            net.deeppoly_bounds_host(w.centers, w.eps)
        assert e.value.code == 6                        # CERT_ERR_TIMEOUT
        lb, ub = net.deeppoly_bounds_host(w.centers, w.eps)
        g["lb"], g["ub"] = lb, ub
        compare(g, ref, label="pm300/host/after a timed-out wait")
    finally:
        net.destroy()


# ---- residual connections (cert_net_create_residual) ----

RES_NETS = {
    "resfc_small": lambda: wl.residual_fc(20, 24, 2, 5, batch=3, eps=0.03, seed=21),
    "resfc_ragged": lambda: wl.residual_fc(50, 70, 3, 7, batch=5, eps=0.02, seed=22),
    "resfc_wide": lambda: wl.residual_fc(64, 300, 2, 10, batch=4, eps=0.01, seed=23),
    "resconv": lambda: wl.residual_conv((2, 10, 8), 4, 2, 6, batch=3, eps=0.02, seed=24),
    "resconv_wide": lambda: wl.residual_conv((3, 16, 16), 8, 1, 10, batch=2, eps=0.01, seed=25),
    # map rows of 64 floats everywhere: the dense conv steps take the banded tensor-core form
    "resconv_band": lambda: wl.residual_conv((4, 16, 16), 8, 2, 10, batch=3, eps=0.01, seed=29),
}


@pytest.mark.parametrize("mode", ["ffma", "tc", "tc16", "auto"])
@pytest.mark.parametrize("name", sorted(RES_NETS))
def test_residual_nets(name, mode):
    w = RES_NETS[name]()
    all_fc = all(l.kind == "fc" for l in w.layers)
    if mode == "tc16" and not all_fc:
        pytest.skip("the fp16 split covers FC nets")
    ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    g = run_gpu(w, contraction={"ffma": 1, "tc": 2, "tc16": 3, "auto": 0}[mode], max_batch=w.batch + 1)
    if mode == "tc16":
        assert g["paths"] & 16 and not g["paths"] & 32      # one launch per back-step, not the chain kernel
    if mode == "auto":
        # FC nets with connections: every layer in the fp16 split on trial; conv nets: the TF32 split
        assert bool(g["paths"] & 128) == all_fc and bool(g["paths"] & 16) == all_fc
    if mode == "tc":
        assert bool(g["paths"] & 64) == (name == "resconv_band")
    compare(g, ref, label=f"{name}/{mode}")
    # the connections matter: the same layers without them give other bounds
    plain = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    assert np.abs(plain["lb"] - g["lb"]).max() > 1e-3


@pytest.mark.parametrize("mode", ["ffma", "tc", "tc16"])
def test_residual_connection_into_the_output_layer_and_back_to_back_blocks(mode):
    w = wl.small_fc([12, 16, 16, 16, 16, 16], batch=3, eps=0.04, seed=26)
    w.skip_from = [-1, -1, 0, -1, 2]        # layer 2 adds layer 0's outputs; the output layer adds layer 2's
    ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    compare(run_gpu(w, contraction={"ffma": 1, "tc": 2, "tc16": 3}[mode]), ref, label=f"output_connection/{mode}")


@pytest.mark.parametrize("mode", ["ffma", "tc"])
@pytest.mark.parametrize("name", ["resfc_ragged", "resfc_wide", "resconv", "resconv_band"])
def test_residual_nets_traversals_that_stop_early(name, mode):
    """IBP, CROWN-IBP, DeepPoly_p and mixed depths: a traversal may end on a connection's source (the waiting
    coefficients join before the simplification), above it (they are simplified on their own), or below it."""
    w = RES_NETS[name]()
    for vname, steps in _variant_steps(len(w.layers)).items():
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                           backsteps_per_layer=steps)
        g = run_gpu(w, contraction=MODES[mode], backsteps=steps)
        compare(g, ref, label=f"{name}/{vname}/{mode}")
    for p in (3, 4):
        steps = [p] * len(w.layers)
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                           backsteps_per_layer=steps)
        compare(run_gpu(w, contraction=MODES[mode], backsteps=steps), ref, label=f"{name}/p{p}/{mode}")


def test_residual_refusals():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.residual_fc(10, 12, 1, 3, batch=2, eps=0.02, seed=27)
    # not two layers back; widths differ; a connection that starts inside another's span
    w5 = wl.small_fc([10, 12, 12, 12, 12, 3], batch=2, eps=0.02, seed=28)
    for layers, bad in ((w.layers, [-1, 0, -1, -1]), (w.layers, [-1, -1, -1, 1]), (w5.layers, [-1, -1, -1, 0, 2])):
        with pytest.raises(binding.CertError):
            binding.CertNet(layers, 2, skip_from=bad)
    net = binding.CertNet(w.layers, 2, skip_from=w.skip_from)
    try:
        assert binding.lib.cert_net_set_conv_patches(net._h, 1) == 2          # CERT_ERR_UNSUPPORTED
        assert binding.lib.cert_net_enable_reusecert(net._h) == 2
        c = torch.from_numpy(w.centers).cuda()
        net.set_contraction(3)
        with pytest.raises(binding.CertError):
            net.backsub_bounds(c, w.eps, [1] * len(w.layers))                  # fp16 split: full traversals only
        net.backsub_bounds(c, w.eps, [-1] * len(w.layers))
        torch.cuda.synchronize()
    finally:
        net.destroy()


# ---- seeded sweep over shapes: every kernel family against the oracle on nets nobody tuned for ----

def _random_fc(seed):
    rng = np.random.default_rng(1000 + seed)
    depth = int(rng.integers(2, 7))
    sizes = [int(rng.integers(3, 90))] + [int(rng.integers(2, 300)) for _ in range(depth)] + [int(rng.integers(1, 12))]
    w = wl.small_fc(sizes, batch=int(rng.integers(1, 6)), eps=float(rng.uniform(0.005, 0.05)), seed=200 + seed)
    if rng.random() < 0.3:
        w.layers[int(rng.integers(0, len(w.layers) - 1))].relu_after = False
    return w


def _random_conv(seed):
    rng = np.random.default_rng(2000 + seed)
    shape = (int(rng.integers(1, 4)), int(rng.integers(8, 17)), int(rng.integers(8, 17)))
    convs, h, wd = [], shape[1], shape[2]
    for _ in range(int(rng.integers(1, 4))):
        k, s = int(rng.integers(2, 5)), int(rng.integers(1, 3))
        p = int(rng.integers(0, min(2, k - 1) + 1))
        ho, wo = (h + 2 * p - k) // s + 1, (wd + 2 * p - k) // s + 1
        if ho < 2 or wo < 2:
            break
        convs.append((int(rng.integers(2, 9)), k, s, p))
        h, wd = ho, wo
    fcs = [int(rng.integers(4, 24)) for _ in range(int(rng.integers(1, 3)))]
    return wl.small_conv(shape, convs, fcs, batch=int(rng.integers(1, 4)), eps=float(rng.uniform(0.005, 0.03)),
                         seed=300 + seed)


def _well_conditioned(make, seed):
    """The net of `seed`, or of seed + 100, + 200, ... if too few of its boxes have branch decisions that float32
    can reproduce (the bump is printed: it is part of the test's record)."""
    from parity_util import MARGIN_MIN
    for bump in range(6):
        w = make(seed + 100 * bump)
        ref = _oracle(w)
        good = ref["margins"].min(axis=1) >= MARGIN_MIN if ref["margins"].shape[1] else np.ones(w.batch, bool)
        if good.mean() >= 0.5:
            print(f"seed {seed}: bump {bump}")
            return w, ref
    raise AssertionError("no well-conditioned net found")


@pytest.mark.parametrize("seed", range(10))
def test_random_fc_shapes_all_contractions(seed):
    w, ref = _well_conditioned(_random_fc, seed)
    for mode, contraction in (("ffma", 1), ("tc", 2), ("tc16", TC16), ("auto", 0)):
        compare(run_gpu(w, contraction=contraction, max_batch=w.batch + (seed % 3)), ref, min_good_fraction=0.5,
                label=f"random_fc[{seed}]/{mode}")


@pytest.mark.parametrize("seed", range(8))
def test_random_conv_shapes(seed):
    w, ref = _well_conditioned(_random_conv, seed)
    for form, kw in (("auto", {}), ("dense", {"conv_patches": False}), ("ffma", {"contraction": 1})):
        compare(run_gpu(w, **kw), ref, min_good_fraction=0.5, label=f"random_conv[{seed}]/{form}")


# ---- a bounded wait that runs out: status word, host mapping, and the net stays usable ----

def test_bounded_wait_runs_out_and_the_net_stays_usable():
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([16, 24, 24, 5], batch=2, eps=0.02, seed=91)
    ref = _oracle(w)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        assert net.last_status() == 0
        net.selftest_bounded_wait()                  # waits about 0.1 ms on a barrier nothing arrives on
        assert net.last_status() == 6                # CERT_ERR_TIMEOUT, read after the stream has drained
        assert net.last_status() == 0                # the read cleared it
        c = torch.from_numpy(w.centers).cuda()
        lb, ub = net.deeppoly_bounds(c, w.eps)
        torch.cuda.synchronize()
        g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": net.branch_codes(w.batch).cpu().numpy(),
             "status": net.last_status(), "layers": w.layers}
        compare(g, ref, label="after a timed-out wait")
    finally:
        net.destroy()


# ---- the call allocates nothing and synchronises nothing: it can be captured into a CUDA graph ----

@pytest.mark.parametrize("mode", ["tc", "tc16", "auto_on_trial"])
def test_call_is_capturable_in_a_cuda_graph(mode):
    import torch
    from paper_2507_20055_b200 import binding
    if mode == "auto_on_trial":
        w = wl.make_config(2, batch=6)           # 784 -> 200 x 9 -> 10: AUTO runs the last layers on trial (a memset
    else:                                        # and predicated re-runs inside the call)
        w = wl.make_config(1, batch=8)           # 784 -> 100 x 6 -> 10
    ref = _oracle(w)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        net.set_contraction({"tc": 2, "tc16": 3, "auto_on_trial": 0}[mode])
        c = torch.from_numpy(w.centers).cuda()
        lb = torch.zeros((w.batch, net.n_total), dtype=torch.float32, device="cuda")
        ub = torch.zeros_like(lb)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            net.deeppoly_bounds(c, w.eps, lb_out=lb, ub_out=ub, stream=s)      # warm-up outside the capture
        s.synchronize()
        lb.zero_(); ub.zero_()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            net.deeppoly_bounds(c, w.eps, lb_out=lb, ub_out=ub, stream=s)
        assert float(lb.abs().max()) == 0.0      # capturing ran nothing
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g = {"lb": lb.cpu().numpy(), "ub": ub.cpu().numpy(), "codes": net.branch_codes(w.batch).cpu().numpy(),
             "status": net.last_status(), "layers": w.layers}
        if mode == "auto_on_trial":
            assert net.last_contraction_paths() & 128
        compare(g, ref, label=f"graph replay/{mode}")
    finally:
        net.destroy()


# ---- fixed summation order: two runs give the same bits ----

@pytest.mark.parametrize("case", ["fc_tc", "fc_tc16", "fc_chain", "conv", "residual"])
def test_results_are_bit_reproducible(case):
    import torch
    from paper_2507_20055_b200 import binding
    if case == "conv":
        w = wl.make_config(3, batch=6)
    elif case == "residual":
        w = wl.residual_fc(64, 300, 2, 10, batch=5, eps=0.01, seed=97)
    elif case == "fc_chain":
        w = wl.make_config(1, batch=16)
    else:
        w = wl.small_fc([200, 700, 700, 700, 10], batch=12, eps=0.01, seed=98)
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    try:
        net.set_contraction({"fc_tc": 2, "fc_tc16": 3, "fc_chain": 3, "conv": 0, "residual": 2}[case])
        c = torch.from_numpy(w.centers).cuda()
        runs = []
        for _ in range(3):
            lb, ub = net.deeppoly_bounds(c, w.eps)
            torch.cuda.synchronize()
            runs.append((lb.clone(), ub.clone()))
        assert net.last_status() == 0
        for lb, ub in runs[1:]:
            assert torch.equal(lb, runs[0][0]) and torch.equal(ub, runs[0][1])
    finally:
        net.destroy()


@pytest.mark.parametrize("block", range(4))
def test_random_nets_with_random_traversal_depths(block):
    """Five FC, three conv and three residual nets per block, every contraction mode that takes them, one random
    traversal depth per affine layer."""
    rng = np.random.default_rng(4000 + block)
    cases = [("fc", _random_fc(30 + 5 * block + i)) for i in range(5)] + \
            [("conv", _random_conv(30 + 3 * block + i)) for i in range(3)]
    for i in range(3):
        r = np.random.default_rng(700 + 3 * block + i)
        cases.append(("res", wl.residual_fc(int(r.integers(5, 60)), int(r.integers(8, 300)), int(r.integers(1, 4)),
                                            int(r.integers(1, 9)), batch=int(r.integers(1, 5)), eps=0.02,
                                            seed=800 + 3 * block + i)))
    for kind, w in cases:
        K = len(w.layers)
        steps = [int(x) for x in rng.integers(-1, K, size=K)]
        ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                           backsteps_per_layer=steps)
        good = ref["margins"].min(axis=1) >= 1e-5 if ref["margins"].shape[1] else np.ones(w.batch, bool)
        if good.mean() < 0.5:
            continue                      # ill-conditioned branch decisions: not a parity case
        modes = {"fc": (1, 2, 3, 0), "conv": (1, None), "res": (1, 2, 0)}[kind]
        for c in modes:
            g = run_gpu(w, contraction=c, backsteps=steps, max_batch=w.batch + block % 2)
            compare(g, ref, label=f"{kind}/{w.name}/mode {c}/depths {steps}")


_BAND_GEOMETRIES = [((2, 16, 16), (4, 8, 12)), ((4, 16, 16), (4, 8)), ((1, 32, 32), (2, 4)), ((4, 8, 8), (8, 16)),
                    ((3, 32, 32), (2, 4))]


@pytest.mark.parametrize("seed", range(6))
def test_random_residual_conv_nets_in_the_banded_form(seed):
    """Residual conv nets whose map rows are multiples of 32 floats (the dense conv steps take the banded
    tensor-core form, the joining step its own kernel variant): one to three blocks, some with the first block's
    connection removed; full traversals and one random depth per layer; FMA and tensor-core modes."""
    r = np.random.default_rng(900 + seed)
    shape, channels = _BAND_GEOMETRIES[int(r.integers(len(_BAND_GEOMETRIES)))]

    def make(s):
        w = wl.residual_conv(shape, int(r.choice(channels)), int(r.integers(1, 4)), int(r.integers(2, 11)),
                             batch=int(r.integers(1, 5)), eps=0.01, seed=1000 + s)
        if seed % 3 == 0 and len(w.layers) > 4:
            w.skip_from = [-1 if k == 2 else s_ for k, s_ in enumerate(w.skip_from)]
        return w

    w, ref = _well_conditioned(make, seed)
    K = len(w.layers)
    steps = [int(x) for x in r.integers(-1, K + 1, size=K)]
    ref_steps = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, skip_from=w.skip_from,
                             backsteps_per_layer=steps)
    for mode, contraction in (("ffma", 1), ("tc", 2)):
        g = run_gpu(w, contraction=contraction, max_batch=w.batch + seed % 2)
        assert bool(g["paths"] & 64) == (mode == "tc")
        compare(g, ref, min_good_fraction=0.5, label=f"residual_band[{seed}]/{mode}")
        compare(run_gpu(w, contraction=contraction, backsteps=steps), ref_steps, min_good_fraction=0.5,
                label=f"residual_band[{seed}]/{mode}/depths {steps}")
