"""ctypes front end of the float64 DeepPoly oracle (TEST INFRASTRUCTURE).

Only tests, the smoke check and the benchmark's CPU-baseline leg use this.
It builds oracle/deeppoly_oracle.c with gcc on first use and calls it; it
imports nothing from the CUDA package.  `layers` is any sequence of objects
with attributes kind ('fc' | 'conv'), weight, bias, relu_after and, for conv,
stride, pad, in_shape (the seeded generators produce such objects).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "deeppoly_oracle.c")
_LIB = os.path.join(_HERE, "libdeeppoly_oracle.so")
_lib = None


class _LayerC(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("kind", "relu_after", "in_features", "out_features",
                 "c_in", "h_in", "w_in", "c_out", "kh", "kw", "stride", "pad")] + \
               [("weight", ctypes.c_void_p), ("bias", ctypes.c_void_p)]


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_deeppoly.restype = ctypes.c_int
        _lib.oracle_backsub.restype = ctypes.c_int
        _lib.oracle_reusecert.restype = ctypes.c_int
        _lib.oracle_num_neurons.restype = ctypes.c_int
        _lib.oracle_num_relu_neurons.restype = ctypes.c_int
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _marshal(layers):
    arr = (_LayerC * len(layers))()
    keep = []
    for i, l in enumerate(layers):
        w = np.ascontiguousarray(l.weight, dtype=np.float32)
        b = np.ascontiguousarray(l.bias, dtype=np.float32)
        keep += [w, b]
        c = arr[i]
        c.relu_after = int(bool(l.relu_after))
        c.weight = w.ctypes.data
        c.bias = b.ctypes.data
        if l.kind == "fc":
            c.kind = 0
            c.out_features, c.in_features = w.shape
        elif l.kind == "conv":
            c.kind = 1
            c.c_out, c.c_in, c.kh, c.kw = w.shape
            _, c.h_in, c.w_in = l.in_shape
            c.stride, c.pad = int(l.stride), int(l.pad)
        else:
            raise ValueError(l.kind)
    return arr, keep


def deeppoly(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, decision_fp32=True,
             max_backsteps: int = -1, n_threads: Optional[int] = None, backsteps_per_layer=None,
             skip_form: bool = False, skip_from=None):
    """Bounds of every affine neuron for every box.

    max_backsteps = p >= 0 is DeepPoly_p; backsteps_per_layer (one count per affine layer,
    negative = traverse to the input) overrides it.  skip_form: the SkipPoly listing (ReLU shapes
    expressed over the neurons two layers back).  skip_from (one entry per affine layer, -1 = none): residual
    connections, layer k adds the outputs of layer skip_from[k] to its affine result.
    Returns dict(lb, ub: float64 [batch, n_total]; codes: uint8 [batch, n_relu];
    margins: float64 [batch, n_relu]).  Layers are concatenated in order.
    """
    lib = _load()
    arr, keep = _marshal(layers)
    centers = np.ascontiguousarray(centers, dtype=np.float32)
    batch = centers.shape[0]
    n_total = lib.oracle_num_neurons(arr, len(layers))
    n_relu = lib.oracle_num_relu_neurons(arr, len(layers))
    lb = np.empty((batch, n_total), dtype=np.float64)
    ub = np.empty((batch, n_total), dtype=np.float64)
    codes = np.empty((batch, n_relu), dtype=np.uint8)
    margins = np.empty((batch, n_relu), dtype=np.float64)
    steps = None
    if backsteps_per_layer is not None:
        steps = np.ascontiguousarray(backsteps_per_layer, dtype=np.int32)
        assert steps.shape == (len(layers),)
    skips = None
    if skip_from is not None:
        skips = np.ascontiguousarray(skip_from, dtype=np.int32)
        assert skips.shape == (len(layers),)
    rc = lib.oracle_backsub(arr, ctypes.c_int(len(layers)), ctypes.c_void_p(centers.ctypes.data),
                            ctypes.c_float(eps), ctypes.c_int(batch), ctypes.c_float(clip_lo),
                            ctypes.c_float(clip_hi), ctypes.c_int(int(decision_fp32)),
                            ctypes.c_int(max_backsteps),
                            ctypes.c_void_p(steps.ctypes.data if steps is not None else None),
                            ctypes.c_int(int(bool(skip_form))),
                            ctypes.c_void_p(skips.ctypes.data if skips is not None else None),
                            ctypes.c_int(n_threads or 0),
                            ctypes.c_void_p(lb.ctypes.data), ctypes.c_void_p(ub.ctypes.data),
                            ctypes.c_void_p(codes.ctypes.data), ctypes.c_void_p(margins.ctypes.data))
    if rc != 0:
        raise RuntimeError(f"oracle_backsub failed with code {rc}")
    del keep
    return {"lb": lb, "ub": ub, "codes": codes, "margins": margins}


def ibp(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, **kw):
    """IBP listing of Appendix C: no traversal at any layer."""
    return deeppoly(layers, centers, eps, clip_lo, clip_hi, backsteps_per_layer=[0] * len(layers), **kw)


def reusecert(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, decision_fp32=True,
              n_threads: Optional[int] = None):
    """ReuseCert listing of Appendix C (bounds kept over the input layer and reused); same outputs as deeppoly()."""
    lib = _load()
    arr, keep = _marshal(layers)
    centers = np.ascontiguousarray(centers, dtype=np.float32)
    batch = centers.shape[0]
    n_total = lib.oracle_num_neurons(arr, len(layers))
    n_relu = lib.oracle_num_relu_neurons(arr, len(layers))
    lb = np.empty((batch, n_total), dtype=np.float64)
    ub = np.empty((batch, n_total), dtype=np.float64)
    codes = np.empty((batch, n_relu), dtype=np.uint8)
    margins = np.empty((batch, n_relu), dtype=np.float64)
    rc = lib.oracle_reusecert(arr, ctypes.c_int(len(layers)), ctypes.c_void_p(centers.ctypes.data),
                              ctypes.c_float(eps), ctypes.c_int(batch), ctypes.c_float(clip_lo),
                              ctypes.c_float(clip_hi), ctypes.c_int(int(decision_fp32)),
                              ctypes.c_int(n_threads or 0),
                              ctypes.c_void_p(lb.ctypes.data), ctypes.c_void_p(ub.ctypes.data),
                              ctypes.c_void_p(codes.ctypes.data), ctypes.c_void_p(margins.ctypes.data))
    if rc != 0:
        raise RuntimeError(f"oracle_reusecert failed with code {rc}")
    del keep
    return {"lb": lb, "ub": ub, "codes": codes, "margins": margins}


def skippoly(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, **kw):
    """SkipPoly listing of Appendix C."""
    return deeppoly(layers, centers, eps, clip_lo, clip_hi, skip_form=True, **kw)


def crown_ibp(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, **kw):
    """CROWN-IBP listing of Appendix C: intervals everywhere, back-substitution at the last layer."""
    return deeppoly(layers, centers, eps, clip_lo, clip_hi,
                    backsteps_per_layer=[0] * (len(layers) - 1) + [-1], **kw)
