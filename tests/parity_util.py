"""Helpers shared by the GPU parity tests: run the CUDA library through its
C ABI and compare with the float64 oracle on the same seeded inputs."""
import numpy as np

TOL = 1e-4            # |gpu - oracle| <= TOL * (1 + |oracle|)
MARGIN_MIN = 1e-5     # boxes with a sign test closer to zero than this are ill-conditioned


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
    finally:
        net.destroy()
    return {"lb": lb, "ub": ub, "codes": codes, "status": status, "launches": launches, "paths": paths}


def compare(gpu, ref, boxes=None, min_good_fraction=0.5, label="", tol=TOL):
    """ref: oracle result for the boxes listed in `boxes` (indices into the GPU batch)."""
    assert gpu["status"] == 0, f"device status {gpu['status']}"
    idx = np.arange(ref["lb"].shape[0]) if boxes is None else np.asarray(boxes)
    lb, ub, codes = gpu["lb"][idx], gpu["ub"][idx], gpu["codes"][idx]
    assert np.isfinite(lb).all() and np.isfinite(ub).all()
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
    print(label, report)
    assert code_mismatch == 0, f"{label}: {code_mismatch} branch codes differ"
    assert worst <= tol, f"{label}: scaled error {worst} > {tol}"
    return report
