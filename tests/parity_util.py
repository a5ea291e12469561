"""Helpers shared by the GPU parity tests: run the CUDA library through its
C ABI and compare with the float64 oracle on the same seeded inputs."""
import hashlib
import os

import numpy as np

from oracle.parity_rule import MARGIN_MIN, TOL, comparable_prefix, layer_layout, parity_report  # noqa: F401

_HERE = os.path.dirname(os.path.abspath(__file__))
_CACHE_DIR = os.path.join(_HERE, ".oracle_cache")
_mem_cache = {}


def cached_oracle(w, certifier="deeppoly"):
    """The oracle's result for every box of workload `w`, computed once per process and kept on disk
    (tests/.oracle_cache/, not under version control) under a key made of the oracle's source, the
    workload's arrays and the certifier, so that a change to any of them recomputes it.  Only oracle/ is
    called to fill it.  The large configurations take minutes of host time; every test that needs them
    shares the one run."""
    from oracle import deeppoly_oracle as orc
    h = hashlib.sha256()
    with open(os.path.join(os.path.dirname(_HERE), "oracle", "deeppoly_oracle.c"), "rb") as f:
        h.update(f.read())
    h.update(certifier.encode())
    for l in w.layers:
        h.update(np.ascontiguousarray(l.weight).tobytes())
        h.update(np.ascontiguousarray(l.bias).tobytes())
        h.update(repr((l.kind, bool(l.relu_after), l.stride, l.pad, l.in_shape)).encode())
    h.update(np.ascontiguousarray(w.centers).tobytes())
    h.update(repr((float(w.eps), float(w.clip_lo), float(w.clip_hi), w.skip_from)).encode())
    key = f"{w.name}_{certifier}_{h.hexdigest()[:16]}"
    if key in _mem_cache:
        return _mem_cache[key]
    path = os.path.join(_CACHE_DIR, key + ".npz")
    if os.path.exists(path):
        with np.load(path) as z:
            ref = {k: z[k] for k in ("lb", "ub", "codes", "margins")}
    else:
        fn = {"deeppoly": orc.deeppoly, "reusecert": orc.reusecert}[certifier]
        kw = {"skip_from": w.skip_from} if certifier == "deeppoly" else {}
        ref = fn(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi, **kw)
        try:
            os.makedirs(_CACHE_DIR, exist_ok=True)
            np.savez(path + ".tmp.npz", **ref)
            os.replace(path + ".tmp.npz", path)
        except OSError:
            pass
    _mem_cache[key] = ref
    return ref


def run_gpu(w, contraction=None, max_batch=None, host_api=False, backsteps=None, conv_patches=None):
    import torch
    from paper_2507_20055_b200 import binding
    net = binding.CertNet(w.layers, max_batch or w.batch, w.clip_lo, w.clip_hi, skip_from=getattr(w, "skip_from", None))
    try:
        if contraction is not None:
            net.set_contraction(contraction)
        if conv_patches is not None:
            net.set_conv_patches(conv_patches)
        if host_api:
            lb, ub = net.deeppoly_bounds_host(w.centers, w.eps)
        else:
            centers = torch.from_numpy(np.ascontiguousarray(w.centers)).cuda()
            if backsteps is None:
                lb_t, ub_t = net.deeppoly_bounds(centers, w.eps)
            else:
                lb_t, ub_t = net.backsub_bounds(centers, w.eps, backsteps)
            torch.cuda.synchronize()
            lb, ub = lb_t.cpu().numpy(), ub_t.cpu().numpy()
        codes = net.branch_codes(w.batch).cpu().numpy()
        status = net.last_status()
        launches = net.last_launch_count()
        paths = net.last_contraction_paths()
        guard = net.check_guards() if hasattr(net, "check_guards") else 0
    finally:
        net.destroy()
    assert guard == 0, f"a guard word around workspace buffer {guard - 1} was overwritten"
    return {"lb": lb, "ub": ub, "codes": codes, "status": status, "launches": launches, "paths": paths,
            "layers": w.layers}


def compare(gpu, ref, boxes=None, min_good_fraction=0.5, label="", tol=TOL, layers=None, min_compared=0.6):
    """ref: oracle result for the boxes listed in `boxes` (indices into the GPU batch).

    With the net's layers known (run_gpu records them; `layers=` otherwise) a box with a near-tie neuron is
    compared up to the layer where the GPU and the oracle resolve a near-tie differently (oracle/parity_rule.py);
    the share of (box, layer) pairs compared must reach min_compared.  Without them a box with any near-tie
    neuron is skipped as a whole."""
    assert gpu["status"] == 0, f"device status {gpu['status']}"
    idx = np.arange(ref["lb"].shape[0]) if boxes is None else np.asarray(boxes)
    lb, ub, codes = gpu["lb"][idx], gpu["ub"][idx], gpu["codes"][idx]
    assert np.isfinite(lb).all() and np.isfinite(ub).all()
    layers = layers if layers is not None else gpu.get("layers")
    if layers is None:
        if ref["margins"].shape[1] > 0:
            good = ref["margins"].min(axis=1) >= MARGIN_MIN
        else:
            good = np.ones(len(idx), dtype=bool)
        assert good.mean() >= min_good_fraction, f"{label}: too many ill-conditioned boxes {good.mean()}"
        code_mismatch = int((codes[good] != ref["codes"][good]).sum())
        err_l = np.abs(lb[good] - ref["lb"][good]) / (1.0 + np.abs(ref["lb"][good]))
        err_u = np.abs(ub[good] - ref["ub"][good]) / (1.0 + np.abs(ref["ub"][good]))
        worst = max(err_l.max(initial=0.0), err_u.max(initial=0.0))
        report = {"boxes": int(len(idx)), "ill_conditioned": int((~good).sum()), "code_mismatches": code_mismatch,
                  "max_scaled_err": float(worst)}
    else:
        assert lb.shape[1] == ref["lb"].shape[1] == sum(l.n_out for l in layers)
        report = parity_report(lb, ub, codes, ref, layers)
        code_mismatch, worst, share = report["code_mismatches"], report["max_scaled_err"], report["share_compared"]
        assert share >= min_compared, f"{label}: only {share:.2f} of the (box, layer) pairs could be compared"
    print(label, report)
    assert code_mismatch == 0, f"{label}: {code_mismatch} branch codes differ"
    assert worst <= tol, f"{label}: scaled error {worst} > {tol}"
    return report
