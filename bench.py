#!/usr/bin/env python
"""Benchmark: input boxes/sec fully bounded by DeepPoly on B200.

One step = one cert_deeppoly_bounds call over one batch of synthetic boxes
(every layer's back-substitution, concretisation and relaxation).
Prints one JSON line (rank 0).  `--impl reference` times the float64 CPU
oracle on the host cores instead (a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2507_20055_b200 import workloads as wl

# DRAM traffic of the dominant kernel, from the ncu captures summarised under profiles/ (read + written bytes of one
# launch of the ReLU-epilogue contraction on a 32-box case, whose matrices (268 / 537 MB each way) exceed L2, per row
# of the coefficient matrix; traffic grows in proportion to the rows, so a full launch is rows x this figure).
# None for workloads not captured.
NCU_TRAFFIC_BYTES_PER_ROW = {
    ("fc6x1024_b128", "tc"): {"bytes_per_row": (628.547840e6 + 487.951616e6) / 65536.0,
                              "kernel": "gemm_tc_kernel<TC_EPI_RELU, 2>",
                              "source": "profiles/gemm_tc_kernel_fc6x1024.md (32 boxes, scaled by rows)"},
    ("fc6x1024_b128", "tc16"): {"bytes_per_row": (273.501952e6 + 230.443776e6) / 65536.0,
                                "kernel": "gemm_tc16_kernel<TC_EPI_RELU, one pass>",
                                "source": "profiles/gemm_tc16_kernel_fc6x1024.md (32 boxes, scaled by rows)"},
}

METRIC = "input boxes/sec fully bounded (DeepPoly)"
UNIT = "boxes/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")] + [time.perf_counter()])

    def stop(self, window=None):
        """window = (t0, t1) in time.perf_counter() terms: only samples read in it count (the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = self.rows
        if window is not None:
            # a sample is printed up to one period after it was taken
            inside = [r for r in rows if window[0] + 0.05 <= r[-1] <= window[1] + 0.05]
            rows = inside or rows
        for r in rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
                for n, v in zip(names, r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(w, n_boxes, threads=None, backsteps=None, certifier="deeppoly"):
    """Times the oracle, as it stands, on the first n_boxes boxes of the workload."""
    from oracle import deeppoly_oracle as orc
    orc.build()
    cores = threads or orc.max_threads()
    c = w.centers[:n_boxes]
    t0 = time.perf_counter()
    if certifier == "reusecert":
        res = orc.reusecert(w.layers, c, w.eps, w.clip_lo, w.clip_hi, n_threads=cores)
    else:
        res = orc.deeppoly(w.layers, c, w.eps, w.clip_lo, w.clip_hi, n_threads=cores, backsteps_per_layer=backsteps,
                           skip_from=w.skip_from)
    dt = time.perf_counter() - t0
    return {"value": n_boxes / dt, "unit": UNIT, "cores": min(cores, n_boxes), "kind": "oracle",
            "sample": f"first {n_boxes} of {w.batch} boxes of {w.name}, one box per thread, {dt:.1f} s wall"}, dt, res


def certifier_steps(name, n_layers):
    """Traversal depth per affine layer (None = to the input everywhere) for a certifier name."""
    if name in ("deeppoly", "reusecert"):
        return None
    if name == "ibp":
        return [0] * n_layers
    if name == "crown_ibp":
        return [0] * (n_layers - 1) + [-1]
    if name.startswith("deeppoly_p"):
        return [int(name[len("deeppoly_p"):])] * n_layers
    raise SystemExit(f"unknown certifier {name!r}")


def patch_levels(layers, k, j_end):
    """Window sizes [(channels, ph, pw), ...] of conv layer k's rows pushed through layers k-1 .. j_end, or None
    where the library keeps dense maps (a non-conv layer on the way, or a window above half its map)."""
    Lk = layers[k]
    if Lk.kind != "conv":
        return None
    _, c_in, kh, kw = Lk.weight.shape
    lv = [(c_in, kh, kw)]
    if 2 * c_in * kh * kw > Lk.n_in:
        return None
    for j in range(k - 1, j_end - 1, -1):
        Lj = layers[j]
        if Lj.kind != "conv":
            return None
        _, cj, kjh, kjw = Lj.weight.shape
        _, ph, pw = lv[-1]
        nx = (cj, (ph - 1) * Lj.stride + kjh, (pw - 1) * Lj.stride + kjw)
        if 2 * nx[0] * nx[1] * nx[2] > Lj.n_in:
            return None
        lv.append(nx)
    return lv


def backstep_flops_by_class(layers, batch, steps=None, patches=True):
    """Algorithmic flops of one call's back-steps: for every layer k, 2*batch*n_k rows go through the
    earlier layers its traversal reaches; an FC step costs 2*n_j*n_{j-1} per row, a conv step on dense
    coefficient maps 2*n_j*c_in*kh*kw, a conv step on a receptive-field patch 2*(window elements)*c_in*kh*kw."""
    out = {"affine": 0.0, "conv": 0.0}
    for k in range(1, len(layers)):
        rows = 2.0 * batch * layers[k].n_out
        depth = k if steps is None or steps[k] < 0 else min(steps[k], k)
        lv = patch_levels(layers, k, k - depth) if (patches and depth > 0) else None
        for m, j in enumerate(range(k - 1, k - depth - 1, -1)):
            L = layers[j]
            if L.kind == "fc":
                out["affine"] += rows * 2.0 * L.n_out * L.n_in
            else:
                _, c_in, kh, kw = L.weight.shape
                elems = lv[m][0] * lv[m][1] * lv[m][2] if lv else L.n_out
                out["conv"] += rows * 2.0 * elems * c_in * kh * kw
    return out


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import deeppoly_oracle as orc
    orc.build()
    cores = orc.max_threads()
    per = {0: 1, 1: 4 * cores, 2: 2 * cores, 3: cores, 4: cores, 5: 2 * cores, 6: cores}
    n_boxes = min(w.batch, args.ref_boxes or per[args.config])
    if args.config == 4 and not args.ref_boxes:
        n_boxes = max(1, min(cores, 16))          # one box per core, about 11 s per box: every core is busy
    times = []
    for i in range(args.warmup + args.steps):
        base, dt, _ = oracle_sample(w, n_boxes, backsteps=args.backsteps, certifier=args.certifier)
        if i >= args.warmup:
            times.append(dt)
    ms = 1000.0 * sum(times) / len(times)
    val = n_boxes / (ms / 1000.0)
    base["value"] = val
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "certifier": args.certifier, "boxes_per_step": n_boxes, "eps": w.eps,
                   "note": "each step bounds a sample of the workload's boxes on the host cores"},
        "cpu_baseline": base,
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4,
                    help="0..4: index into the benchmark configurations; 5: a fully connected residual net in the "
                         "shape of the paper's 'Skip' network (784 -> 512 x 5 -> 10, two blocks, 64 boxes); 6: a residual "
                         "conv net (3x32x32 -> conv16 s2 -> two blocks of two 3x3 convs -> 10, 16 boxes)")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--contraction", default="auto", choices=["auto", "ffma", "tc", "tc16"],
                    help="auto = what the plain three-call ABI runs (the fp16 split where the net's weights prove its "
                         "range, else 3xTF32); tc = tcgen05 3xTF32, tc16 = tcgen05 fp16 split (FC nets), ffma = FMA units")
    ap.add_argument("--certifier", default="deeppoly",
                    help="deeppoly | ibp | crown_ibp | deeppoly_pN (N back-substitution steps per layer) | reusecert")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-microbench", action="store_true", help="skip the peak micro-kernels (roofline against the bf16-derived peaks only)")
    ap.add_argument("--ref-boxes", type=int, default=None)
    args = ap.parse_args()

    if args.config == 5:
        w = wl.residual_fc(784, 512, 2, 10, batch=args.batch or 64, eps=0.01, seed=0)
    elif args.config == 6:
        w = wl.residual_conv((3, 32, 32), 16, 2, 10, batch=args.batch or 16, eps=2.0 / 255.0, seed=0)
    else:
        w = wl.make_config(args.config, batch=args.batch)
    args.backsteps = certifier_steps(args.certifier, len(w.layers))
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2507_20055_b200 import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.warmup < 3:
        args.warmup = 3
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2507_20055_b200 import binding

    # Boxes are independent: the job's boxes (per-GPU batch x ranks: weak scaling) are split with
    # box_shard, the weights are replicated, and there is no collective on the data path.
    if world > 1:
        from paper_2507_20055_b200 import sharding
        per_gpu = w.batch
        everything = wl.centers_uniform(per_gpu * world, w.centers.shape[1], seed=0)
        w.centers = sharding.shard_centers(everything, rank, world)
        assert w.batch == per_gpu
    B = w.batch
    net = binding.CertNet(w.layers, B, w.clip_lo, w.clip_hi, skip_from=w.skip_from)
    mode = {"auto": binding.CONTRACTION_AUTO, "ffma": binding.CONTRACTION_FFMA, "tc": binding.CONTRACTION_TC3XTF32,
            "tc16": binding.CONTRACTION_TC3XFP16}
    net.set_contraction(mode[args.contraction])
    resolved = args.contraction
    if args.contraction == "auto":
        resolved = {1: "ffma", 2: "tc", 3: "tc16"}[net.auto_contraction()]
    stream = torch.cuda.Stream()
    centers = torch.from_numpy(w.centers).cuda()
    lb = torch.empty((B, net.n_total), dtype=torch.float32, device="cuda")
    ub = torch.empty_like(lb)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # > 126 MB L2
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    reuse = args.certifier == "reusecert"
    if reuse:
        net.enable_reusecert()

    def step_device():
        if reuse:
            net.reusecert_bounds(centers, w.eps, lb, ub, stream=stream)
        else:
            net.backsub_bounds(centers, w.eps, args.backsteps, lb, ub, stream=stream)

    # ---- device-resident timing: K steps, each bracketed by events on the launching stream,
    #      L2 flushed between steps outside the bracket ----
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step_device()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    t_wall0 = time.perf_counter()
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            flush.fill_(i & 0xFF)
            evs[i][0].record(stream)
            step_device()
            evs[i][1].record(stream)
    barrier()
    t_wall1 = time.perf_counter()
    t_wall = t_wall1 - t_wall0
    step_ms = [a.elapsed_time(b) for a, b in evs]
    total_ms = sum(step_ms)
    launches = net.last_launch_count() * args.steps
    assert net.last_status(stream.cuda_stream) == 0, "device-side status is not OK"

    # ---- per-kernel-class times over the same K steps (events inside the library) ----
    net.set_profiling(True)
    cls_ms, cls_n = {}, {}
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            flush.fill_(i & 0xFF)
            step_device()
            stream.synchronize()
            for name, (ms, n) in net.profile().items():
                cls_ms[name] = cls_ms.get(name, 0.0) + ms
                cls_n[name] = cls_n.get(name, 0) + n
    net.set_profiling(False)
    clocks = sampler.stop((t_wall0, t_wall1)) if rank == 0 else None

    # ---- the same steps with the 3xTF32 contraction, for reference, when the fp16 split was timed above ----
    tf32_ref = None
    if resolved == "tc16" and world == 1 and not reuse:
        net.set_contraction(binding.CONTRACTION_TC3XTF32)
        n_ref = max(3, min(args.steps, 5))
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ref)]
        with torch.cuda.stream(stream):
            for _ in range(3):
                step_device()
            for i in range(n_ref):
                flush.fill_(i & 0xFF)
                ev2[i][0].record(stream)
                step_device()
                ev2[i][1].record(stream)
        stream.synchronize()
        ms_ref = sum(a.elapsed_time(b) for a, b in ev2) / n_ref
        tf32_ref = {"value": B / (ms_ref / 1000.0), "unit": UNIT, "ms_per_step": ms_ref, "steps": n_ref,
                    "contraction": "tc (3xTF32)"}
        assert net.last_status(stream.cuda_stream) == 0
        net.set_contraction(mode[args.contraction])

    # ---- end to end through the host-buffer entry point (pinned buffers, copies timed) ----
    centers_pin = torch.from_numpy(w.centers).pin_memory()
    lb_pin = torch.empty((B, net.n_total), dtype=torch.float32).pin_memory()
    ub_pin = torch.empty((B, net.n_total), dtype=torch.float32).pin_memory()
    c_np, lb_np, ub_np = centers_pin.numpy(), lb_pin.numpy(), ub_pin.numpy()

    def step_host():
        if reuse:
            net.reusecert_bounds_host(c_np, w.eps, lb_np, ub_np, stream.cuda_stream)
        else:
            net.deeppoly_bounds_host(c_np, w.eps, lb_np, ub_np, stream.cuda_stream, args.backsteps)

    for _ in range(2):
        step_host()
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()   # returns after the D2H copy
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    # ---- the denominators, measured: micro-kernels that run nothing but the unit in question.  They run in a
    #      child process with a time limit: whatever happens there cannot stall or fail the benchmark line (the
    #      roofline then falls back to the bf16-derived peak) ----
    micro = None
    if rank == 0 and world == 1 and not args.no_microbench:
        torch.cuda.synchronize()
        code = ("import json\nfrom paper_2507_20055_b200 import binding\nout = {}\n"
                "for name, kind in (('tcgen05_f16', 0), ('tcgen05_tf32', 1), ('ffma', 2)):\n"
                "    try:\n"
                "        b = binding.peak_microbench(kind, 5.0)\n"
                "        s = binding.peak_microbench(kind, 250.0)\n"
                "        out[name] = {'burst': {'tflops': b[0], 'sm_mhz': b[1], 'ms': b[2]},\n"
                "                     'sustained': {'tflops': s[0], 'sm_mhz': s[1], 'ms': s[2]}}\n"
                "    except binding.CertError as e:\n"
                "        out[name] = {'error': str(e)}\n"
                "try:\n"
                "    t = binding.peak_microbench(3, 5.0)\n"
                "    out['tma_l2_to_smem'] = {'tb_per_s': t[0], 'sm_mhz': t[1], 'ms': t[2],\n"
                "                             'bytes_per_cycle_per_sm': t[0] * 1e12 / (t[1] * 1e6) / %d}\n"
                "except binding.CertError as e:\n"
                "    out['tma_l2_to_smem'] = {'error': str(e)}\n"
                "print('MICRO ' + json.dumps(out))\n" % torch.cuda.get_device_properties(local_rank).multi_processor_count)
        try:
            env = dict(os.environ, CUDA_VISIBLE_DEVICES=os.environ.get("CUDA_VISIBLE_DEVICES", str(local_rank)))
            r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True,
                               timeout=120)
            lines = [x for x in r.stdout.splitlines() if x.startswith("MICRO ")]
            micro = json.loads(lines[-1][6:]) if lines else {"error": (r.stderr or "no output")[-300:]}
        except subprocess.TimeoutExpired:
            micro = {"error": "the micro-kernels did not finish within 120 s"}
        except Exception as e:          # noqa: BLE001  (the benchmark line must come out whatever happens here)
            micro = {"error": repr(e)[:300]}

    # ---- max over ranks ----
    t = torch.tensor([total_ms, e2e_s * 1000.0], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms_max, e2e_ms_max = float(t[0]), float(t[1])
    value = world * B * args.steps / (total_ms_max / 1000.0)
    e2e_value = world * B * e2e_steps / (e2e_ms_max / 1000.0)

    if rank == 0:
        peaks = load_peaks()
        used_patches = bool(net.last_contraction_paths() & 8)
        fl = backstep_flops_by_class(w.layers, B, args.backsteps, patches=used_patches)
        fl_dense = backstep_flops_by_class(w.layers, B, args.backsteps, patches=False)
        if reuse:
            # one contraction per affine layer k >= 1: (n0 + 1) rows per box (coefficients and the constant),
            # 2 n_{k-1} columns of shapes below against the 2 n_k shapes of the layer
            n0 = w.layers[0].n_in
            fl = {"affine": sum(2.0 * B * (n0 + 1) * (2 * l.n_in) * (2 * l.n_out) for l in w.layers[1:]), "conv": 0.0}
            fl_dense = fl
        flops_call = fl["affine"] + fl["conv"]
        if args.backsteps is None and not reuse:      # the library's own count (dense maps) must agree
            lib_count = net.backstep_flops(B)
            assert abs(fl_dense["affine"] + fl_dense["conv"] - lib_count) <= 1e-6 * lib_count
        # the dominant kernel class: FC back-steps (tensor cores unless --contraction ffma) or conv back-steps (FMA units)
        dom = "affine" if cls_ms.get("affine", 0.0) >= cls_ms.get("conv", 0.0) else "conv"
        dom_ms, dom_n = cls_ms.get(dom, 0.0), cls_n.get(dom, 0)
        achieved = fl[dom] * args.steps / (dom_ms / 1000.0) / 1e12 if dom_ms > 0 else None
        sm_max = (clocks or {}).get("sm_max_mhz") or 1965.0
        ffma_peak = 148 * 128 * 2 * sm_max * 1e6 / 1e12
        # fp32-accurate work on the tensor cores costs three TF32 products per multiply-add;
        # TF32 dense peak = measured bf16 (sustained: the kernel runs inside a long step) x 1/2 (nominal ratio)
        used_fp16 = bool(net.last_contraction_paths() & 16)
        # fp16 split: three fp16 products (bf16 rate) per multiply-add; TF32 split: three TF32 products (half that rate)
        tc_peak = peaks["bf16_tflops_sustained"] * (1.0 if used_fp16 else 0.5) / 3.0
        # conv back-steps: on the tensor cores when the dense steps ran in banded form (bit 6) beside the patch steps
        used_tc = bool(net.last_contraction_paths() & 2) and (dom == "affine" or bool(net.last_contraction_paths() & 64))
        traffic, traffic_note = None, "no ncu capture for this workload / contraction mode"
        cap = NCU_TRAFFIC_BYTES_PER_ROW.get((w.name, "tc16" if used_fp16 else "tc"))
        if cap and used_tc and (net.last_contraction_paths() & 4) and not reuse and args.backsteps is None:
            rows_per_launch = 2.0 * B * max(l.n_out for l in w.layers[1:-1] or w.layers[1:])
            traffic = cap["bytes_per_row"] * rows_per_launch
            traffic_note = f"{cap['kernel']}: {cap['source']}"
        derived_peak = tc_peak if used_tc else ffma_peak
        peak, peak_source, frac_same_clock = derived_peak, peaks["source"], None
        pipe = ("tcgen05_f16" if used_fp16 else "tcgen05_tf32") if used_tc else "ffma"
        m = (micro or {}).get(pipe)
        if m and "sustained" in m:
            # the pipe's own measured rate, under the power limit like the timed step; a fp32-accurate
            # multiply-add costs three products on the tensor cores
            div = 3.0 if used_tc else 1.0
            peak = m["sustained"]["tflops"] / div
            peak_source = "microbench"
            clk = (clocks or {}).get("sm_mhz")
            if achieved and clk and m["sustained"]["sm_mhz"]:
                frac_same_clock = (achieved / clk) / (peak / m["sustained"]["sm_mhz"])
        if used_tc:
            derived_note = "bf16_tflops_sustained/3 (3xFP16)" if used_fp16 else "bf16_tflops_sustained/2/3 (3xTF32)"
            if dom == "conv":
                derived_note += ("; conv back-steps run as dense window / band contractions, counted here at their "
                                 "algorithmic flops (the executed count is several times higher)")
        else:
            derived_note = "148 SM x 128 FMA x 2 x sm_max_mhz"
            if used_patches and args.contraction != "ffma":
                derived_note += ("; the conv class also holds the patch back-step, which runs on the tensor cores "
                                 "(gather + 3xTF32 contraction with the window-to-window matrix), counted at its "
                                 "algorithmic flops")
        peak_note = derived_note
        if peak_source == "microbench":
            peak_note = (f"microbench: {pipe} sustained" + (" / 3" if used_tc else "") +
                         "; peak_bf16_derived = " + derived_note)
        roof = {"bound": "tensor" if used_tc else "alu",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved / peak) if achieved else None,
                "frac_same_clock": frac_same_clock,
                "peak_bf16_derived": derived_peak,
                "frac_bf16_derived": (achieved / derived_peak) if achieved else None,
                "peak_bf16_derived_source": peaks["source"],
                "traffic": traffic, "traffic_note": traffic_note,
                "kernel": dom + " back-step", "launches_per_step": dom_n // max(1, args.steps),
                "avg_launch_ms": dom_ms / dom_n if dom_n else None,
                "flops_per_step": fl[dom], "flops_per_step_all_backsteps": flops_call,
                "flops_per_step_if_dense_maps": fl_dense[dom], "conv_rows_as_patches": used_patches,
                "peak_source": peak_source,
                "peak_note": peak_note,
                "class_ms_per_step": {k: v / args.steps for k, v in cls_ms.items()}}
        # branch statistics of the last call (Relu transformer): the share of ReLU neurons relaxed as unstable
        torch.cuda.synchronize()
        codes = net.branch_codes(B)
        torch.cuda.synchronize()
        unstable = float((codes >= 2).float().mean().item()) if codes.numel() else 0.0
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "certifier": args.certifier, "boxes_per_gpu": B, "eps": w.eps,
                       "net": "->".join(str(x) for x in [w.layers[0].n_in] + [l.n_out for l in w.layers]),
                       "contraction": args.contraction, "contraction_resolved": resolved, "parallelism": f"replicas over boxes x{world}",
                       "l2": "256 MiB flush write between timed steps; per-step coefficient traffic exceeds L2"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(B * net.n0 * 4),
                    "d2h_bytes_per_step": int(2 * B * net.n_total * 4), "steps": e2e_steps},
            "gpu_launches": launches, "wall_s_timed_region": t_wall, "roofline": roof, "clocks": clocks,
            "unstable_fraction": unstable,
        }
        if micro is not None:
            out["peaks_microbench"] = micro
        if tf32_ref is not None:
            out["tf32_split"] = tf32_ref
        if world == 1 and not args.no_cpu_baseline:
            n_boxes = {0: 1, 1: 64, 2: 32, 3: 16, 4: 16, 5: 32, 6: 16}[args.config]
            from oracle import deeppoly_oracle as orc
            orc.build()
            n_boxes = min(n_boxes, B) if args.config != 4 else min(B, orc.max_threads(), 16)
            out["cpu_baseline"], _, ref = oracle_sample(w, n_boxes, backsteps=args.backsteps, certifier=args.certifier)
            if args.config in (0, 1):
                one, _, _ = oracle_sample(w, min(n_boxes, 4), threads=1, backsteps=args.backsteps,
                                          certifier=args.certifier)
                out["cpu_baseline"]["single_thread"] = {"value": one["value"], "unit": UNIT, "sample": one["sample"]}
            # parity of the timed configuration: the bounds of the last timed device call against the oracle
            # boxes just computed (same rule and tolerance as the tests: oracle/parity_rule.py)
            from oracle import parity_rule
            with torch.cuda.stream(stream):
                step_device()
            stream.synchronize()
            rep = parity_rule.parity_report(lb[:n_boxes].cpu().numpy(), ub[:n_boxes].cpu().numpy(),
                                            net.branch_codes(B)[:n_boxes].cpu().numpy(), ref, w.layers)
            rep["tolerance"] = parity_rule.TOL
            rep["ok"] = bool(rep["code_mismatches"] == 0 and rep["max_scaled_err"] <= parity_rule.TOL)
            out["parity"] = rep
        print(json.dumps(out))
    net.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
