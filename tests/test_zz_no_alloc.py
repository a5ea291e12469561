"""The allocation-free entry point against the regular one and against the oracle.

cert_first_layer_bounds_noalloc serves embedders that cannot allocate device memory (they live
inside another framework's memory pool, or have a fixed budget); it must give the same interval
bounds as cert_deeppoly_bounds on a one-layer net, and both must match the float64 oracle's bounds
of that net.  It keeps its scratch in an array shared by all
calls, so the check runs two calls in a row with different inputs: the second must not see anything
of the first.  Collected last on purpose, so that a run stopping at the first failure has already
run every other test.
"""
import numpy as np
import pytest

from oracle import deeppoly_oracle as orc
from paper_2507_20055_b200 import workloads as wl
from parity_util import TOL

pytestmark = pytest.mark.gpu


def _regular(w):
    import torch
    from paper_2507_20055_b200 import binding
    net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
    try:
        lb, ub = net.deeppoly_bounds(torch.from_numpy(w.centers).cuda(), w.eps)
        torch.cuda.synchronize()
        return lb.cpu().numpy(), ub.cpu().numpy()
    finally:
        net.destroy()


def test_noalloc_matches_regular_entry_point_twice():
    import torch
    from paper_2507_20055_b200 import binding
    first = wl.small_fc([784, 300], batch=37, eps=0.03, seed=81)
    second = wl.small_fc([50, 21], batch=5, eps=0.2, seed=82)     # smaller: stale scratch lies beyond it
    for w in (first, second):
        ref_lb, ref_ub = _regular(w)
        oracle = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
        layer = w.layers[0]
        weight = torch.from_numpy(layer.weight).cuda()
        bias = torch.from_numpy(layer.bias).cuda()
        centers = torch.from_numpy(w.centers).cuda()
        lb = torch.full((w.batch, layer.n_out), float("nan"), device="cuda")
        ub = torch.full((w.batch, layer.n_out), float("nan"), device="cuda")
        binding.first_layer_bounds_noalloc(weight, bias, centers, w.eps, w.clip_lo, w.clip_hi, lb, ub)
        torch.cuda.synchronize()
        lb, ub = lb.cpu().numpy(), ub.cpu().numpy()
        assert np.isfinite(lb).all() and np.isfinite(ub).all()
        assert (np.abs(lb - ref_lb) <= TOL * (1 + np.abs(ref_lb))).all()
        assert (np.abs(ub - ref_ub) <= TOL * (1 + np.abs(ref_ub))).all()
        assert (np.abs(lb - oracle["lb"]) <= TOL * (1 + np.abs(oracle["lb"]))).all()
        assert (np.abs(ub - oracle["ub"]) <= TOL * (1 + np.abs(oracle["ub"]))).all()


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2507_20055_b200 import binding
    weight = torch.zeros((4, 1024), device="cuda")
    bias = torch.zeros(4, device="cuda")
    centers = torch.zeros((1025, 1024), device="cuda")       # 1025 * 1024 floats > 2^20
    lb = torch.zeros((1025, 4), device="cuda")
    ub = torch.zeros((1025, 4), device="cuda")
    with pytest.raises(binding.CertError) as e:
        binding.first_layer_bounds_noalloc(weight, bias, centers, 0.1, 0.0, 1.0, lb, ub)
    assert e.value.code == 4
    rc = binding.lib.cert_first_layer_bounds_noalloc(None, bias.data_ptr(), 4, 1024, centers.data_ptr(), 0.1,
                                                     0.0, 1.0, 1, lb.data_ptr(), ub.data_ptr(), None)
    assert rc == 1


def test_noalloc_allocates_no_device_memory():
    """Free device memory as the driver reports it is the same before and after a (warm) call."""
    import torch
    from paper_2507_20055_b200 import binding
    w = wl.small_fc([64, 40], batch=8, eps=0.05, seed=83)
    layer = w.layers[0]
    weight, bias = torch.from_numpy(layer.weight).cuda(), torch.from_numpy(layer.bias).cuda()
    centers = torch.from_numpy(w.centers).cuda()
    lb = torch.empty((w.batch, layer.n_out), device="cuda")
    ub = torch.empty_like(lb)
    binding.first_layer_bounds_noalloc(weight, bias, centers, w.eps, w.clip_lo, w.clip_hi, lb, ub)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        binding.first_layer_bounds_noalloc(weight, bias, centers, w.eps, w.clip_lo, w.clip_hi, lb, ub)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
