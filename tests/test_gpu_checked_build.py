"""The checking build of the library (-DCERT_BOUNDS): every plain global store of the kernels that do not go
through TMA is looked up in a table of the buffers the call may write, and a store outside all of them is skipped
and reported.  compute-sanitizer is not available here; this build and the guard words around every buffer
(cert_net_check_guards, checked after every run_gpu) stand in for it.  The library is loaded once per process, so
the checking build runs in child processes (CERT_LIB selects it)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _env():
    from paper_2507_20055_b200 import build
    return dict(os.environ, CERT_LIB=build.build_checked(), CERT_EXPECT_CHECKED="1")


def test_ordinary_build_has_no_checked_stores():
    import torch  # noqa: F401
    from paper_2507_20055_b200 import binding, workloads as wl
    if os.environ.get("CERT_LIB"):
        pytest.skip("running against another build")
    assert binding.lib.cert_built_with_checked_stores() == 0
    w = wl.small_fc([8, 8, 4], batch=2, eps=0.1, seed=77)
    net = binding.CertNet(w.layers, 2)
    try:
        assert binding.lib.cert_net_selftest_checked_store(net._h, None) == 2      # CERT_ERR_UNSUPPORTED
    finally:
        net.destroy()


_SELFTEST = r"""
import numpy as np, torch
from paper_2507_20055_b200 import binding, workloads as wl
from oracle import deeppoly_oracle as orc
assert binding.lib.cert_built_with_checked_stores() == 1
w = wl.small_fc([33, 64, 64, 10], batch=4, eps=0.04, seed=75)
net = binding.CertNet(w.layers, w.batch, w.clip_lo, w.clip_hi)
c = torch.from_numpy(w.centers).cuda()
lb, ub = net.deeppoly_bounds(c, w.eps)
torch.cuda.synchronize()
assert net.last_status() == 0
net.selftest_checked_store()                 # a store one float past the box array: refused, nothing written
assert net.last_status() == 8                # CERT_ERR_BOUNDS
assert net.last_status() == 0
assert net.check_guards() == 0               # the guard bytes it aimed at are intact
lb2, ub2 = net.deeppoly_bounds(c, w.eps)
torch.cuda.synchronize()
assert net.last_status() == 0 and torch.equal(lb, lb2) and torch.equal(ub, ub2)
ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
assert (np.abs(lb.cpu().numpy() - ref["lb"]) <= 1e-4 * (1 + np.abs(ref["lb"]))).all()
net.destroy()
print("selftest ok")
"""


def test_checked_build_refuses_a_store_outside_every_buffer():
    r = subprocess.run([sys.executable, "-c", _SELFTEST], env=_env(), cwd=ROOT, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0 and "selftest ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_checked_build_runs_the_sweeps_without_a_refused_store():
    """The parity sweeps on small shapes (every kernel family, ragged batches, bounded traversals, residual nets,
    ReuseCert) under the checking build: a refused store would come back as status 8 and fail the comparison."""
    select = ("small_and_ragged or random_fc_shapes or random_conv_shapes or test_residual_nets or "
              "test_bounded_traversals or test_conv_rows or banded or batch_smaller or missing_relu or "
              "(test_reusecert and not config5) or (fp16_split and not config5) or random_nets_with_random")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x",
                        "-m", "gpu", "-k", select, "-p", "no:cacheprovider"],
                       env=_env(), cwd=ROOT, capture_output=True, text=True, timeout=3000)
    tail = r.stdout[-3000:] + r.stderr[-1000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout.splitlines()[-1], tail
