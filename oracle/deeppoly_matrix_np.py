"""Second, structurally different float64 DeepPoly (TEST INFRASTRUCTURE).

Where the C oracle walks one neuron's expression at a time with scalar sign
tests, this file uses the layer-level form the paper's rewrites arrive at
(Section 4.3: the Matmul rewrite turns map(c*n[L]) into a matrix product, the
ternary/clamp rewrites turn `c >= 0 ? c*L : c*U` into
clamp(c, min=0)*L + clamp(c, max=0)*U).  Conv layers are expanded to dense
matrices by index arithmetic.  It exists to cross-check the C oracle; it
imports neither the C oracle nor the CUDA package.
"""
from __future__ import annotations

import numpy as np


def dense_matrix(layer) -> np.ndarray:
    """[n_out, n_in] float64 matrix of an affine layer (conv: cross-correlation, zero padding)."""
    w = np.asarray(layer.weight, dtype=np.float64)
    if layer.kind == "fc":
        return w
    c_out, c_in, kh, kw = w.shape
    _, h, wd = layer.in_shape
    s, p = layer.stride, layer.pad
    ho, wo = (h + 2 * p - kh) // s + 1, (wd + 2 * p - kw) // s + 1
    m = np.zeros((c_out, ho, wo, c_in, h, wd), dtype=np.float64)
    oy, ox = np.meshgrid(np.arange(ho), np.arange(wo), indexing="ij")
    for ky in range(kh):
        for kx in range(kw):
            iy, ix = oy * s - p + ky, ox * s - p + kx
            ok = (iy >= 0) & (iy < h) & (ix >= 0) & (ix < wd)
            for co in range(c_out):
                for ci in range(c_in):
                    m[co, oy[ok], ox[ok], ci, iy[ok], ix[ok]] = w[co, ci, ky, kx]
    return m.reshape(c_out * ho * wo, c_in * h * wd)


def dense_bias(layer) -> np.ndarray:
    b = np.asarray(layer.bias, dtype=np.float64)
    if layer.kind == "fc":
        return b
    n_out = dense_matrix_rows(layer)
    return np.repeat(b, n_out // b.shape[0])


def dense_matrix_rows(layer) -> int:
    if layer.kind == "fc":
        return layer.weight.shape[0]
    c_out, _, kh, kw = layer.weight.shape
    _, h, wd = layer.in_shape
    s, p = layer.stride, layer.pad
    return c_out * ((h + 2 * p - kh) // s + 1) * ((wd + 2 * p - kw) // s + 1)


def box(centers, eps, clip_lo, clip_hi):
    c = np.asarray(centers, dtype=np.float32)
    e = np.float32(eps)
    l0 = np.maximum(c - e, np.float32(clip_lo)).astype(np.float64)
    u0 = np.minimum(c + e, np.float32(clip_hi)).astype(np.float64)
    return l0, u0


def deeppoly_matrix(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, decision_fp32=True, backsteps=None,
                    skip_from=None):
    """Returns lb, ub [batch, n_total] float64 and codes [batch, n_relu] uint8.

    backsteps: optional list with one traversal-step count per affine layer (negative: to the
    input).  A traversal that stops early is simplified against the concrete bounds of the
    neurons it reached (Section 6.2, DeepPoly_p; 0 everywhere is the IBP listing, 0 except at
    the last layer the CROWN-IBP listing of Appendix C).
    skip_from: optional residual connections (layer k adds the outputs of layer skip_from[k]): the
    coefficient matrix on those outputs is set aside and joins the expression when the traversal, highest
    layer first, has come down to that layer; if the traversal stops before, it is simplified against
    that layer's concrete bounds."""
    A = [dense_matrix(l) for l in layers]
    bias = [dense_bias(l) for l in layers]
    L0, U0 = box(centers, eps, clip_lo, clip_hi)
    batch = L0.shape[0]
    n_total = sum(a.shape[0] for a in A)
    n_relu = sum(a.shape[0] for a, l in zip(A, layers) if l.relu_after)
    lb_all = np.empty((batch, n_total))
    ub_all = np.empty((batch, n_total))
    codes_all = np.empty((batch, n_relu), dtype=np.uint8)
    for b in range(batch):
        l0, u0 = L0[b], U0[b]
        lam_l, lam_u, nu_u = [], [], []
        act_l, act_u = [], []       # concrete bounds of each layer's outputs (after its ReLU, if any)
        off, coff = 0, 0
        for k, layer in enumerate(layers):
            Cl, Cu = A[k].copy(), A[k].copy()
            dl, du = bias[k].copy(), bias[k].copy()
            limit = -1 if backsteps is None else int(backsteps[k])
            stop_at = -1 if limit < 0 else max(k - 1 - limit, -1)   # layer whose outputs the expression ends on
            waiting = {}
            if skip_from is not None and skip_from[k] >= 0:
                eye = np.eye(A[k].shape[0])
                waiting[skip_from[k]] = (eye, eye.copy())
            for j in range(k - 1, stop_at, -1):
                if j in waiting:
                    Wl, Wu = waiting.pop(j)
                    Cl, Cu = Cl + Wl, Cu + Wu
                if layers[j].relu_after:
                    Clp, Clm = np.clip(Cl, 0.0, None), np.clip(Cl, None, 0.0)
                    Cup, Cum = np.clip(Cu, 0.0, None), np.clip(Cu, None, 0.0)
                    dl = dl + Clm @ nu_u[j]
                    du = du + Cup @ nu_u[j]
                    Cl = Clp * lam_l[j] + Clm * lam_u[j]
                    Cu = Cup * lam_u[j] + Cum * lam_l[j]
                if skip_from is not None and skip_from[j] >= 0:
                    Wl, Wu = waiting.get(skip_from[j], (0.0, 0.0))
                    waiting[skip_from[j]] = (Wl + Cl, Wu + Cu)
                dl = dl + Cl @ bias[j]
                du = du + Cu @ bias[j]
                Cl = Cl @ A[j]
                Cu = Cu @ A[j]
            if stop_at >= 0 and stop_at in waiting:
                Wl, Wu = waiting.pop(stop_at)
                Cl, Cu = Cl + Wl, Cu + Wu
            lo_in, up_in = (l0, u0) if stop_at < 0 else (act_l[stop_at], act_u[stop_at])
            lb = np.clip(Cl, 0.0, None) @ lo_in + np.clip(Cl, None, 0.0) @ up_in + dl
            ub = np.clip(Cu, 0.0, None) @ up_in + np.clip(Cu, None, 0.0) @ lo_in + du
            for t2, (Wl, Wu) in waiting.items():      # neurons of lower layers still in the expression
                lb = lb + np.clip(Wl, 0.0, None) @ act_l[t2] + np.clip(Wl, None, 0.0) @ act_u[t2]
                ub = ub + np.clip(Wu, 0.0, None) @ act_u[t2] + np.clip(Wu, None, 0.0) @ act_l[t2]
            n_k = lb.shape[0]
            if layer.relu_after:
                act_l.append(np.maximum(lb, 0.0)); act_u.append(np.maximum(ub, 0.0))
            else:
                act_l.append(lb); act_u.append(ub)
            lb_all[b, off:off + n_k], ub_all[b, off:off + n_k] = lb, ub
            off += n_k
            if layer.relu_after:
                if decision_fp32:
                    lf, uf = lb.astype(np.float32), ub.astype(np.float32)
                    active, inactive, pick = lf >= 0, uf <= 0, (lf + uf) >= 0
                else:
                    active, inactive, pick = lb >= 0, ub <= 0, (lb + ub) >= 0
                unstable = ~active & ~inactive
                den = np.where(unstable, ub - lb, 1.0)
                lam_u.append(np.where(active, 1.0, np.where(inactive, 0.0, ub / den)))
                nu_u.append(np.where(unstable, -(ub * lb) / den, 0.0))
                lam_l.append(np.where(pick, 1.0, 0.0))
                codes_all[b, coff:coff + n_k] = np.where(active, 1, np.where(inactive, 0, 2 + pick))
                coff += n_k
            else:
                lam_l.append(None); lam_u.append(None); nu_u.append(None)
    return lb_all, ub_all, codes_all


def reusecert_matrix(layers, centers, eps, clip_lo=0.0, clip_hi=1.0, decision_fp32=True):
    """ReuseCert (Appendix C listing) in layer-level form: the shapes of every layer's outputs are kept as
    matrices over the input, [coefficients | constant], and an affine layer composes them with its sign-split
    weights: L_k = W+ L_below + W- U_below + b, U_k = W+ U_below + W- L_below + b (clamp form of Section 4.3).
    Returns lb, ub [batch, n_total] and codes [batch, n_relu]."""
    A = [dense_matrix(l) for l in layers]
    bias = [dense_bias(l) for l in layers]
    L0, U0 = box(centers, eps, clip_lo, clip_hi)
    batch, n0 = L0.shape
    n_total = sum(a.shape[0] for a in A)
    n_relu = sum(a.shape[0] for a, l in zip(A, layers) if l.relu_after)
    lb_all, ub_all = np.empty((batch, n_total)), np.empty((batch, n_total))
    codes_all = np.empty((batch, n_relu), dtype=np.uint8)
    for b in range(batch):
        l0, u0 = L0[b], U0[b]
        off = coff = 0
        Lb = Ub = None                       # [n, n0 + 1]: last column is the constant
        for k, layer in enumerate(layers):
            Wp, Wm = np.clip(A[k], 0.0, None), np.clip(A[k], None, 0.0)
            if k == 0:
                Lk = Uk = np.concatenate([A[0], bias[0][:, None]], axis=1)
            else:
                Lk = Wp @ Lb + Wm @ Ub
                Uk = Wp @ Ub + Wm @ Lb
                Lk[:, -1] += bias[k]
                Uk[:, -1] += bias[k]
            lb = np.clip(Lk[:, :n0], 0.0, None) @ l0 + np.clip(Lk[:, :n0], None, 0.0) @ u0 + Lk[:, -1]
            ub = np.clip(Uk[:, :n0], 0.0, None) @ u0 + np.clip(Uk[:, :n0], None, 0.0) @ l0 + Uk[:, -1]
            n_k = lb.shape[0]
            lb_all[b, off:off + n_k], ub_all[b, off:off + n_k] = lb, ub
            off += n_k
            if layer.relu_after:
                if decision_fp32:
                    lf, uf = lb.astype(np.float32), ub.astype(np.float32)
                    active, inactive, pick = lf >= 0, uf <= 0, (lf + uf) >= 0
                else:
                    active, inactive, pick = lb >= 0, ub <= 0, (lb + ub) >= 0
                unstable = ~active & ~inactive
                den = np.where(unstable, ub - lb, 1.0)
                lam_u = np.where(active, 1.0, np.where(inactive, 0.0, ub / den))
                nu_u = np.where(unstable, -(ub * lb) / den, 0.0)
                lam_l = np.where(pick, 1.0, 0.0)
                Lb = lam_l[:, None] * Lk
                Ub = lam_u[:, None] * Uk
                Ub[:, -1] += nu_u
                codes_all[b, coff:coff + n_k] = np.where(active, 1, np.where(inactive, 0, 2 + pick))
                coff += n_k
            else:
                Lb, Ub = Lk.copy(), Uk.copy()
    return lb_all, ub_all, codes_all


def forward_preactivations(layers, x):
    """Plain float64 forward pass; x [m, n0]; returns [m, n_total] pre-activations."""
    A = [dense_matrix(l) for l in layers]
    bias = [dense_bias(l) for l in layers]
    a = np.asarray(x, dtype=np.float64)
    outs = []
    for k, layer in enumerate(layers):
        z = a @ A[k].T + bias[k]
        outs.append(z)
        a = np.maximum(z, 0.0) if layer.relu_after else z
    return np.concatenate(outs, axis=1)
