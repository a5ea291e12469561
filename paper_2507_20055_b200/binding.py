"""Thin ctypes binding of libcert_b200.so (argument marshalling only).

Every step of the path runs in the library's CUDA kernels.  PyTorch is used
for device memory and streams.  There is no CPU fallback: if the library is
missing or cannot be loaded, import of this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# CERT_LIB selects another build of the same library (the checking build of build.py), for tests
LIB_PATH = os.environ.get("CERT_LIB") or os.path.join(_HERE, "libcert_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2507_20055_b200.build` "
        "(nvcc, sm_100a); there is no CPU fallback")

_lib = ctypes.CDLL(LIB_PATH)

CERT_OK = 0
CONTRACTION_AUTO, CONTRACTION_FFMA, CONTRACTION_TC3XTF32, CONTRACTION_TC3XFP16 = 0, 1, 2, 3

EXPORTS = [
    "cert_net_create", "cert_net_create_residual", "cert_deeppoly_bounds", "cert_backsub_bounds", "cert_deeppoly_bounds_host",
    "cert_backsub_bounds_host",
    "cert_net_destroy",
    "cert_net_num_neurons", "cert_net_num_relu_neurons", "cert_net_branch_codes",
    "cert_net_last_status", "cert_net_selftest_bounded_wait", "cert_net_set_contraction", "cert_net_last_launch_count",
    "cert_net_backstep_flops", "cert_status_string", "cert_net_set_profiling", "cert_net_profile",
    "cert_net_last_contraction_paths", "cert_first_layer_bounds_noalloc", "cert_net_set_conv_patches",
    "cert_net_enable_reusecert", "cert_reusecert_bounds", "cert_reusecert_bounds_host",
    "cert_net_check_guards", "cert_net_auto_contraction", "cert_net_fp16_coefficient_bound",
    "cert_peak_microbench", "cert_built_with_checked_stores", "cert_net_selftest_checked_store",
]
CLASS_NAMES = ["input", "relax", "relu_step", "affine", "conv", "concretize"]


class cert_layer_desc_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("kind", "relu_after", "in_features", "out_features",
                 "c_in", "h_in", "w_in", "c_out", "kh", "kw", "stride", "pad")] + \
               [("weight", ctypes.c_void_p), ("bias", ctypes.c_void_p)]


_vp, _i, _f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
_lib.cert_net_create.argtypes = [ctypes.POINTER(cert_layer_desc_t), _i, _i, _f, _f, ctypes.POINTER(_vp)]
_lib.cert_net_create.restype = _i
_lib.cert_net_create_residual.argtypes = [ctypes.POINTER(cert_layer_desc_t), _i, _vp, _i, _f, _f, ctypes.POINTER(_vp)]
_lib.cert_net_create_residual.restype = _i
_lib.cert_deeppoly_bounds.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp]
_lib.cert_deeppoly_bounds.restype = _i
_lib.cert_backsub_bounds.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp, _vp]
_lib.cert_backsub_bounds.restype = _i
_lib.cert_backsub_bounds_host.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp, _vp]
_lib.cert_backsub_bounds_host.restype = _i
_lib.cert_deeppoly_bounds_host.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp]
_lib.cert_deeppoly_bounds_host.restype = _i
_lib.cert_net_destroy.argtypes = [_vp]
_lib.cert_net_destroy.restype = _i
_lib.cert_net_num_neurons.argtypes = [_vp]
_lib.cert_net_num_neurons.restype = _i
_lib.cert_net_num_relu_neurons.argtypes = [_vp]
_lib.cert_net_num_relu_neurons.restype = _i
_lib.cert_net_branch_codes.argtypes = [_vp, _vp, _vp]
_lib.cert_net_branch_codes.restype = _i
_lib.cert_net_last_status.argtypes = [_vp, _vp]
_lib.cert_net_last_status.restype = _i
_lib.cert_net_selftest_bounded_wait.argtypes = [_vp, _vp]
_lib.cert_net_selftest_bounded_wait.restype = _i
_lib.cert_net_set_contraction.argtypes = [_vp, _i]
_lib.cert_net_set_contraction.restype = _i
_lib.cert_net_last_launch_count.argtypes = [_vp]
_lib.cert_net_last_launch_count.restype = _i
_lib.cert_net_backstep_flops.argtypes = [_vp, _i]
_lib.cert_net_backstep_flops.restype = ctypes.c_double
_lib.cert_net_last_contraction_paths.argtypes = [_vp]
_lib.cert_net_last_contraction_paths.restype = _i
_lib.cert_net_enable_reusecert.argtypes = [_vp]
_lib.cert_net_enable_reusecert.restype = _i
_lib.cert_reusecert_bounds.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp]
_lib.cert_reusecert_bounds.restype = _i
_lib.cert_reusecert_bounds_host.argtypes = [_vp, _vp, _f, _i, _vp, _vp, _vp]
_lib.cert_reusecert_bounds_host.restype = _i
_lib.cert_net_set_conv_patches.argtypes = [_vp, _i]
_lib.cert_net_set_conv_patches.restype = _i
_lib.cert_net_set_profiling.argtypes = [_vp, _i]
_lib.cert_net_set_profiling.restype = _i
_lib.cert_net_profile.argtypes = [_vp, _vp, _vp]
_lib.cert_net_profile.restype = _i
_lib.cert_first_layer_bounds_noalloc.argtypes = [_vp, _vp, _i, _i, _vp, _f, _f, _f, _i, _vp, _vp, _vp]
_lib.cert_first_layer_bounds_noalloc.restype = _i
_lib.cert_net_check_guards.argtypes = [_vp, _vp]
_lib.cert_net_check_guards.restype = _i
_lib.cert_net_auto_contraction.argtypes = [_vp]
_lib.cert_net_auto_contraction.restype = _i
_lib.cert_net_fp16_coefficient_bound.argtypes = [_vp, _i]
_lib.cert_net_fp16_coefficient_bound.restype = ctypes.c_float
_lib.cert_built_with_checked_stores.argtypes = []
_lib.cert_built_with_checked_stores.restype = _i
_lib.cert_net_selftest_checked_store.argtypes = [_vp, _vp]
_lib.cert_net_selftest_checked_store.restype = _i
_lib.cert_peak_microbench.argtypes = [_i, ctypes.c_double, _vp, _vp, _vp, _vp]
_lib.cert_peak_microbench.restype = _i
_lib.cert_status_string.argtypes = [_i]
_lib.cert_status_string.restype = ctypes.c_char_p


class CertError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.cert_status_string(code).decode()} (status {code})")


def _check(code: int, where: str):
    if code != CERT_OK:
        raise CertError(code, where)


def marshal_layers(layers: Sequence):
    """ctypes array of cert_layer_desc_t from objects with kind/weight/bias/relu_after(/stride/pad/in_shape)."""
    arr = (cert_layer_desc_t * len(layers))()
    keep = []
    for i, l in enumerate(layers):
        w = np.ascontiguousarray(l.weight, dtype=np.float32)
        b = np.ascontiguousarray(l.bias, dtype=np.float32)
        keep += [w, b]
        d = arr[i]
        d.relu_after = int(bool(l.relu_after))
        d.weight, d.bias = w.ctypes.data, b.ctypes.data
        if l.kind == "fc":
            d.kind = 0
            d.out_features, d.in_features = w.shape
        elif l.kind == "conv":
            d.kind = 1
            d.c_out, d.c_in, d.kh, d.kw = w.shape
            _, d.h_in, d.w_in = l.in_shape
            d.stride, d.pad = int(l.stride), int(l.pad)
        else:
            raise ValueError(f"unknown layer kind {l.kind!r}")
    return arr, keep


def _check_tensor(name, t, shape, device=None):
    """The kernels take raw pointers: a wrong dtype, layout, shape or device would be an out-of-bounds access."""
    import torch
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError(f"{name}: a contiguous float32 CUDA tensor is required")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: shape {tuple(t.shape)}, expected {tuple(shape)}")
    if device is not None and t.device != device:
        raise ValueError(f"{name}: on {t.device}, expected {device}")


class CertNet:
    """Owns a cert_net_t handle; the three calls of the C ABI plus the helpers."""

    def __init__(self, layers: Sequence, max_batch: int, clip_lo: float = 0.0, clip_hi: float = 1.0,
                 skip_from=None):
        """skip_from: residual connections, one entry per layer (-1 = none): cert_net_create_residual."""
        arr, keep = marshal_layers(layers)
        h = _vp()
        if skip_from is None:
            _check(_lib.cert_net_create(arr, len(layers), int(max_batch), float(clip_lo), float(clip_hi),
                                        ctypes.byref(h)), "cert_net_create")
        else:
            assert len(skip_from) == len(layers)
            skips = (ctypes.c_int * len(layers))(*[int(x) for x in skip_from])
            _check(_lib.cert_net_create_residual(arr, len(layers), ctypes.cast(skips, _vp), int(max_batch),
                                                 float(clip_lo), float(clip_hi), ctypes.byref(h)),
                   "cert_net_create_residual")
        self._h = h
        self.max_batch = int(max_batch)
        self.n0 = int(layers[0].n_in)
        self.n_total = int(_lib.cert_net_num_neurons(h))
        self.n_relu = int(_lib.cert_net_num_relu_neurons(h))
        self.n_layers = len(layers)

    # -- raw-pointer form (what the C ABI takes) --
    def deeppoly_bounds_ptr(self, centers_ptr: int, eps: float, batch: int, lb_ptr: int, ub_ptr: int,
                            stream_ptr: int = 0):
        _check(_lib.cert_deeppoly_bounds(self._h, centers_ptr, float(eps), int(batch), lb_ptr, ub_ptr,
                                         stream_ptr), "cert_deeppoly_bounds")

    # -- torch tensors on the device --
    def deeppoly_bounds(self, centers, eps: float, lb_out=None, ub_out=None, stream=None):
        import torch
        batch = centers.shape[0]
        _check_tensor("centers", centers, (batch, self.n0))
        if lb_out is None:
            lb_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        if ub_out is None:
            ub_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        _check_tensor("lb_out", lb_out, (batch, self.n_total), centers.device)
        _check_tensor("ub_out", ub_out, (batch, self.n_total), centers.device)
        st = stream if stream is not None else torch.cuda.current_stream(centers.device)
        self.deeppoly_bounds_ptr(centers.data_ptr(), eps, batch, lb_out.data_ptr(), ub_out.data_ptr(),
                                 st.cuda_stream)
        return lb_out, ub_out

    def backsub_bounds(self, centers, eps: float, backsteps=None, lb_out=None, ub_out=None, stream=None):
        """cert_backsub_bounds: backsteps = one traversal depth per affine layer (negative: to the input)."""
        import torch
        batch = centers.shape[0]
        _check_tensor("centers", centers, (batch, self.n0))
        if lb_out is None:
            lb_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        if ub_out is None:
            ub_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        _check_tensor("lb_out", lb_out, (batch, self.n_total), centers.device)
        _check_tensor("ub_out", ub_out, (batch, self.n_total), centers.device)
        st = stream if stream is not None else torch.cuda.current_stream(centers.device)
        steps = None
        if backsteps is not None:
            assert len(backsteps) == self.n_layers
            steps = (ctypes.c_int * self.n_layers)(*[int(x) for x in backsteps])
        _check(_lib.cert_backsub_bounds(self._h, centers.data_ptr(), float(eps), int(batch),
                                        ctypes.addressof(steps) if steps is not None else None,
                                        lb_out.data_ptr(), ub_out.data_ptr(), st.cuda_stream), "cert_backsub_bounds")
        return lb_out, ub_out

    def enable_reusecert(self):
        _check(_lib.cert_net_enable_reusecert(self._h), "cert_net_enable_reusecert")

    def reusecert_bounds(self, centers, eps: float, lb_out=None, ub_out=None, stream=None):
        """cert_reusecert_bounds (enable_reusecert() first)."""
        import torch
        batch = centers.shape[0]
        _check_tensor("centers", centers, (batch, self.n0))
        if lb_out is None:
            lb_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        if ub_out is None:
            ub_out = torch.empty((batch, self.n_total), dtype=torch.float32, device=centers.device)
        _check_tensor("lb_out", lb_out, (batch, self.n_total), centers.device)
        _check_tensor("ub_out", ub_out, (batch, self.n_total), centers.device)
        st = stream if stream is not None else torch.cuda.current_stream(centers.device)
        _check(_lib.cert_reusecert_bounds(self._h, centers.data_ptr(), float(eps), int(batch), lb_out.data_ptr(),
                                          ub_out.data_ptr(), st.cuda_stream), "cert_reusecert_bounds")
        return lb_out, ub_out

    def reusecert_bounds_host(self, centers: np.ndarray, eps: float, lb: np.ndarray, ub: np.ndarray,
                              stream_ptr: int = 0):
        centers = np.ascontiguousarray(centers, dtype=np.float32)
        _check(_lib.cert_reusecert_bounds_host(self._h, centers.ctypes.data, float(eps), centers.shape[0],
                                               lb.ctypes.data, ub.ctypes.data, stream_ptr),
               "cert_reusecert_bounds_host")
        return lb, ub

    def deeppoly_p_bounds(self, centers, eps: float, p: int, **kw):
        return self.backsub_bounds(centers, eps, [int(p)] * self.n_layers, **kw)

    def ibp_bounds(self, centers, eps: float, **kw):
        return self.backsub_bounds(centers, eps, [0] * self.n_layers, **kw)

    def crown_ibp_bounds(self, centers, eps: float, **kw):
        return self.backsub_bounds(centers, eps, [0] * (self.n_layers - 1) + [-1], **kw)

    # -- host numpy arrays (copies inside the library) --
    def deeppoly_bounds_host(self, centers: np.ndarray, eps: float, lb: Optional[np.ndarray] = None,
                             ub: Optional[np.ndarray] = None, stream_ptr: int = 0, backsteps=None):
        centers = np.ascontiguousarray(centers, dtype=np.float32)
        batch = centers.shape[0]
        if lb is None:
            lb = np.empty((batch, self.n_total), dtype=np.float32)
        if ub is None:
            ub = np.empty((batch, self.n_total), dtype=np.float32)
        steps = None
        if backsteps is not None:
            assert len(backsteps) == self.n_layers
            steps = (ctypes.c_int * self.n_layers)(*[int(x) for x in backsteps])
        _check(_lib.cert_backsub_bounds_host(self._h, centers.ctypes.data, float(eps), batch,
                                             ctypes.addressof(steps) if steps is not None else None,
                                             lb.ctypes.data, ub.ctypes.data, stream_ptr),
               "cert_backsub_bounds_host")
        return lb, ub

    def set_profiling(self, on: bool):
        _check(_lib.cert_net_set_profiling(self._h, int(bool(on))), "cert_net_set_profiling")

    def profile(self):
        """dict class name -> (ms, launches) of the most recent call (profiling must be on)."""
        ms = (ctypes.c_float * len(CLASS_NAMES))()
        cnt = (ctypes.c_int * len(CLASS_NAMES))()
        _check(_lib.cert_net_profile(self._h, ctypes.addressof(ms), ctypes.addressof(cnt)), "cert_net_profile")
        return {n: (float(ms[i]), int(cnt[i])) for i, n in enumerate(CLASS_NAMES)}

    def branch_codes(self, batch: int, stream=None):
        import torch
        if self.n_relu == 0:
            return torch.empty((batch, 0), dtype=torch.uint8, device="cuda")
        codes = torch.empty((batch, self.n_relu), dtype=torch.uint8, device="cuda")
        st = stream if stream is not None else torch.cuda.current_stream()
        _check(_lib.cert_net_branch_codes(self._h, codes.data_ptr(), st.cuda_stream), "cert_net_branch_codes")
        return codes

    def last_status(self, stream_ptr: int = 0) -> int:
        return int(_lib.cert_net_last_status(self._h, stream_ptr))

    def selftest_bounded_wait(self, stream_ptr: int = 0):
        """Enqueues a kernel whose (short) bounded wait runs out; last_status() then reports CERT_ERR_TIMEOUT."""
        _check(_lib.cert_net_selftest_bounded_wait(self._h, stream_ptr), "cert_net_selftest_bounded_wait")

    def set_contraction(self, mode: int):
        _check(_lib.cert_net_set_contraction(self._h, int(mode)), "cert_net_set_contraction")

    def set_conv_patches(self, on: bool):
        _check(_lib.cert_net_set_conv_patches(self._h, int(bool(on))), "cert_net_set_conv_patches")

    def selftest_checked_store(self, stream_ptr: int = 0):
        """Checking build only: one store just past a buffer, which is refused; last_status() then reports 8."""
        _check(_lib.cert_net_selftest_checked_store(self._h, stream_ptr), "cert_net_selftest_checked_store")

    def check_guards(self, stream_ptr: int = 0) -> int:
        """0 = every guard word around the net's device buffers is intact, i + 1 = allocation i was overrun."""
        return int(_lib.cert_net_check_guards(self._h, stream_ptr))

    def auto_contraction(self) -> int:
        return int(_lib.cert_net_auto_contraction(self._h))

    def fp16_coefficient_bound(self, layer: int = -1) -> float:
        return float(_lib.cert_net_fp16_coefficient_bound(self._h, int(layer)))

    def last_contraction_paths(self) -> int:
        return int(_lib.cert_net_last_contraction_paths(self._h))

    def last_launch_count(self) -> int:
        return int(_lib.cert_net_last_launch_count(self._h))

    def backstep_flops(self, batch: int) -> float:
        return float(_lib.cert_net_backstep_flops(self._h, int(batch)))

    def destroy(self):
        if getattr(self, "_h", None):
            _check(_lib.cert_net_destroy(self._h), "cert_net_destroy")
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def first_layer_bounds_noalloc(weight, bias, centers, eps, clip_lo, clip_hi, lb_out, ub_out, stream=None):
    """Interval bounds of one FC layer without any allocation inside the library.

    All tensors are the caller's torch CUDA tensors (float32, contiguous): weight [out, in],
    bias [out], centers [batch, in], lb_out / ub_out [batch, out].  For embedders that may not
    allocate device memory; see cert_first_layer_bounds_noalloc in cert.h for the limit and the
    rules on sharing.  Raises CertError on a bad argument or a batch beyond the built-in limit.
    """
    import torch
    out_features, in_features = weight.shape
    batch = centers.shape[0]
    for name, t, shape in (("weight", weight, (out_features, in_features)), ("bias", bias, (out_features,)),
                           ("centers", centers, (batch, in_features)), ("lb_out", lb_out, (batch, out_features)),
                           ("ub_out", ub_out, (batch, out_features))):
        _check_tensor(name, t, shape, weight.device)
    st = stream if stream is not None else torch.cuda.current_stream(weight.device)
    _check(_lib.cert_first_layer_bounds_noalloc(weight.data_ptr(), bias.data_ptr(), out_features, in_features,
                                                centers.data_ptr(), float(eps), float(clip_lo), float(clip_hi),
                                                centers.shape[0], lb_out.data_ptr(), ub_out.data_ptr(),
                                                st.cuda_stream), "cert_first_layer_bounds_noalloc")


def peak_microbench(kind: int, target_ms: float = 5.0, stream_ptr: int = 0):
    """cert_peak_microbench: (TFLOP/s, SM MHz seen by the kernel, ms) for kind 0 = tcgen05 f16, 1 = tcgen05 tf32,
    2 = fp32 FMA units; kind 3 = bulk copies from L2 into shared memory, first value in TB/s over all SMs."""
    out = (ctypes.c_double * 3)()
    base = ctypes.addressof(out)
    _check(_lib.cert_peak_microbench(int(kind), float(target_ms), base, base + 8, base + 16, stream_ptr),
           "cert_peak_microbench")
    return float(out[0]), float(out[1]), float(out[2])


# C-ABI names, as plain functions
cert_net_create = _lib.cert_net_create
cert_deeppoly_bounds = _lib.cert_deeppoly_bounds
cert_backsub_bounds = _lib.cert_backsub_bounds
cert_deeppoly_bounds_host = _lib.cert_deeppoly_bounds_host
cert_net_destroy = _lib.cert_net_destroy
lib = _lib
