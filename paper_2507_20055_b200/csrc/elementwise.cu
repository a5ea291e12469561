// Bandwidth-bound steps of the DeepPoly path: box construction, first-layer
// interval bounds, ReLU relaxation, start of a back-substitution, the unfused
// ReLU back-step and the unfused concretisation.  One warp owns one row of a
// coefficient matrix; row sums are warp-shuffle trees, so every result is
// deterministic.
#include <algorithm>
#include <cstdlib>

#include "common.cuh"

namespace cert {

namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float tf32_round(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// replace_lower / replace_upper through a ReLU neuron whose bounds are
// L = lamL*z and U = lamU*z + nuU (Appendix C, DeepPoly listing).  Returns the
// coefficient over z and adds the constant part to dacc.
__device__ __forceinline__ float relu_backstep(float c, int upper, float lamL, float lamU, float nuU,
                                               float &dacc) {
    const bool nonneg = (c >= 0.0f);
    const bool use_lower = upper ? !nonneg : nonneg;
    if (use_lower) return c * lamL;
    dacc = fmaf(c, nuU, dacc);
    return c * lamU;
}

__global__ void box_kernel(const float *__restrict__ centers, float eps, float lo, float hi, int batch,
                           int n0, int ld0, float *__restrict__ l0, float *__restrict__ u0) {
    pdl_trigger();
    pdl_wait();
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * ld0) return;
    int b = (int)(idx / ld0), s = (int)(idx % ld0);
    float l = 0.0f, u = 0.0f;
    if (s < n0) {
        float c = centers[(size_t)b * n0 + s];
        l = fmaxf(__fsub_rn(c, eps), lo);
        u = fminf(__fadd_rn(c, eps), hi);
    }
    CERT_ST(l0[idx], l);
    CERT_ST(u0[idx], u);
}

// FC layer: one warp per (box, NEURONS consecutive neurons).  The box row is read once for the warp's neurons
// (the weight rows come from L2 either way); every output is summed lane-strided and reduced by a shuffle tree.
template <int NEURONS>
__global__ void first_layer_kernel(const float *__restrict__ W, const float *__restrict__ bias_n, int n_in, int ld_in,
                                   int n_out, const float *__restrict__ l0, const float *__restrict__ u0, int ld0,
                                   int batch, float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                                   int out_off) {
    pdl_trigger();
    pdl_wait();
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int groups = (n_out + NEURONS - 1) / NEURONS;
    if (warp >= (long long)batch * groups) return;
    const int b = (int)(warp / groups), i0 = (int)(warp % groups) * NEURONS;
    const int n_here = n_out - i0 < NEURONS ? n_out - i0 : NEURONS;
    const float *lrow = l0 + (size_t)b * ld0, *urow = u0 + (size_t)b * ld0;
    const float *w = W + (size_t)i0 * ld_in;
    float lo[NEURONS], hi[NEURONS];
#pragma unroll
    for (int e = 0; e < NEURONS; ++e) lo[e] = hi[e] = 0.0f;
    for (int s = lane; s < n_in; s += 32) {
        const float l = lrow[s], u = urow[s];
#pragma unroll
        for (int e = 0; e < NEURONS; ++e) {
            if (e < n_here) {
                const float c = w[(size_t)e * ld_in + s];
                const bool nn = (c >= 0.0f);
                lo[e] = fmaf(c, nn ? l : u, lo[e]);
                hi[e] = fmaf(c, nn ? u : l, hi[e]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < NEURONS; ++e) {
        const float lo_s = warp_sum(lo[e]), hi_s = warp_sum(hi[e]);
        if (lane == 0 && e < n_here) {
            const float bb = bias_n[i0 + e];
            CERT_ST(lb_out[(size_t)b * n_total + out_off + i0 + e], lo_s + bb);
            CERT_ST(ub_out[(size_t)b * n_total + out_off + i0 + e], hi_s + bb);
        }
    }
}

// The same with 16-byte loads, for rows whose pitches are multiples of four floats and whose padding up to the
// next multiple of four is zero (the net's own arrays; a caller's unpadded weights when in_features % 4 == 0).
template <int NEURONS>
__global__ void first_layer_vec_kernel(const float *__restrict__ W, const float *__restrict__ bias_n, int n_in, int ld_in,
                                       int n_out, const float *__restrict__ l0, const float *__restrict__ u0, int ld0,
                                       int batch, float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                                       int out_off) {
    pdl_trigger();
    pdl_wait();
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int groups = (n_out + NEURONS - 1) / NEURONS;
    if (warp >= (long long)batch * groups) return;
    const int b = (int)(warp / groups), i0 = (int)(warp % groups) * NEURONS;
    const int n_here = n_out - i0 < NEURONS ? n_out - i0 : NEURONS;
    const float4 *lrow = reinterpret_cast<const float4 *>(l0 + (size_t)b * ld0);
    const float4 *urow = reinterpret_cast<const float4 *>(u0 + (size_t)b * ld0);
    float lo[NEURONS], hi[NEURONS];
#pragma unroll
    for (int e = 0; e < NEURONS; ++e) lo[e] = hi[e] = 0.0f;
    const int quads = (n_in + 3) >> 2;
    for (int q = lane; q < quads; q += 32) {
        const float4 l4 = lrow[q], u4 = urow[q];
        const float l[4] = {l4.x, l4.y, l4.z, l4.w}, u[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
        for (int e = 0; e < NEURONS; ++e) {
            if (e < n_here) {
                const float4 w4 = *reinterpret_cast<const float4 *>(W + (size_t)(i0 + e) * ld_in + 4 * q);
                const float c[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int z = 0; z < 4; ++z) {
                    const bool nn = (c[z] >= 0.0f);
                    lo[e] = fmaf(c[z], nn ? l[z] : u[z], lo[e]);
                    hi[e] = fmaf(c[z], nn ? u[z] : l[z], hi[e]);
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < NEURONS; ++e) {
        const float lo_s = warp_sum(lo[e]), hi_s = warp_sum(hi[e]);
        if (lane == 0 && e < n_here) {
            const float bb = bias_n[i0 + e];
            CERT_ST(lb_out[(size_t)b * n_total + out_off + i0 + e], lo_s + bb);
            CERT_ST(ub_out[(size_t)b * n_total + out_off + i0 + e], hi_s + bb);
        }
    }
}

// The same for a conv layer with one thread per (box, neuron): a neuron has only c_in*kh*kw taps, and
// the threads of a warp are neighbouring positions of one channel, so the weights are warp-uniform loads.
__global__ void first_layer_conv_kernel(const float *__restrict__ W, const float *__restrict__ bias_n, ConvGeom g,
                                        int n_out, const float *__restrict__ l0, const float *__restrict__ u0,
                                        int ld0, int batch, float *__restrict__ lb_out,
                                        float *__restrict__ ub_out, int n_total, int out_off) {
    pdl_trigger();
    pdl_wait();
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * n_out) return;
    const int b = (int)(idx / n_out), i = (int)(idx % n_out);
    const float *lrow = l0 + (size_t)b * ld0, *urow = u0 + (size_t)b * ld0;
    const int hw = g.h_out * g.w_out;
    const int co = i / hw, oy = (i / g.w_out) % g.h_out, ox = i % g.w_out;
    const int y0 = oy * g.stride - g.pad, x0 = ox * g.stride - g.pad;
    const float *w = W + (size_t)co * g.c_in * g.kh * g.kw;
    float lo = 0.0f, hi = 0.0f;
    for (int ci = 0; ci < g.c_in; ++ci)
        for (int ky = 0; ky < g.kh; ++ky) {
            const int iy = y0 + ky;
            if (iy < 0 || iy >= g.h_in) continue;
            const int base = (ci * g.h_in + iy) * g.w_in;
            const float *wr = w + (ci * g.kh + ky) * g.kw;
            for (int kx = 0; kx < g.kw; ++kx) {
                const int ix = x0 + kx;
                if (ix < 0 || ix >= g.w_in) continue;
                const float c = wr[kx], l = lrow[base + ix], u = urow[base + ix];
                const bool nn = (c >= 0.0f);
                lo = fmaf(c, nn ? l : u, lo);
                hi = fmaf(c, nn ? u : l, hi);
            }
        }
    const float bb = bias_n[i];
    CERT_ST(lb_out[(size_t)b * n_total + out_off + i], lo + bb);
    CERT_ST(ub_out[(size_t)b * n_total + out_off + i], hi + bb);
}

// Joins the waiting coefficients of a residual connection to the expression that has reached its source.
__global__ void add_skip_kernel(float *__restrict__ P, const float *__restrict__ S_hi,
                                const float *__restrict__ S_lo, int identity, long long total, int n, int ld,
                                int n_k) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const long long r = idx / ld;
    const int t = (int)(idx - r * ld);
    if (t >= n) return;
    float s = 0.0f;
    if (S_hi) s = S_hi[idx] + (S_lo ? S_lo[idx] : 0.0f);
    if (identity && t == (int)(r % n_k)) s += 1.0f;
    CERT_ST(P[idx], (P[idx]) + (s));
}

// Interval step of a layer with a residual connection: the source's concrete output bounds are added.
__global__ void add_act_bounds_kernel(float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                                      int out_off, int n_k, int batch, const float *__restrict__ actL,
                                      const float *__restrict__ actU, int ld_act) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * n_k) return;
    const int b = (int)(idx / n_k), i = (int)(idx % n_k);
    CERT_ST(lb_out[(size_t)b * n_total + out_off + i], (lb_out[(size_t)b * n_total + out_off + i]) + (actL[(size_t)b * ld_act + i]));
    CERT_ST(ub_out[(size_t)b * n_total + out_off + i], (ub_out[(size_t)b * n_total + out_off + i]) + (actU[(size_t)b * ld_act + i]));
}

// A traversal stopped with coefficients still waiting on a residual connection's source: those neurons are
// simplified against their own concrete bounds (map(simplify_lower/upper)); one warp per row.  The term goes
// to a slot of the row constants (slot != nullptr) or is added to the bounds already written.
__global__ void skip_concretize_kernel(const float *__restrict__ S_hi, const float *__restrict__ S_lo, int identity,
                                       const float *__restrict__ actL, const float *__restrict__ actU, int ld_act,
                                       long long rows, int n, int ld, int n_k, float *__restrict__ slot,
                                       float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                                       int out_off) {
    const long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const int b = (int)(r / (2LL * n_k));
    const int upper = (int)((r / n_k) & 1);
    const int i = (int)(r % n_k);
    const float *lrow = actL + (size_t)b * ld_act, *urow = actU + (size_t)b * ld_act;
    float term = 0.0f;
    if (S_hi) {
        for (int t = lane; t < n; t += 32) {
            float c = S_hi[(size_t)r * ld + t];
            if (S_lo) c += S_lo[(size_t)r * ld + t];
            const bool nonneg = (c >= 0.0f);
            term = fmaf(c, (nonneg != (upper != 0)) ? lrow[t] : urow[t], term);
        }
        term = warp_sum(term);
    }
    if (lane == 0) {
        if (identity) term += upper ? urow[i] : lrow[i];
        if (slot) CERT_ST(slot[r], term);
        else CERT_ST((upper ? ub_out : lb_out)[(size_t)b * n_total + out_off + i], ((upper ? ub_out : lb_out)[(size_t)b * n_total + out_off + i]) + (term));
    }
}

// Sum of the slots that hold a row's constant (or bound), in slot order.
__device__ __forceinline__ float slot_sum(const float *__restrict__ d, int n_slots, long long stride,
                                          long long r) {
    float v = d[r];
    for (int s = 1; s < n_slots; ++s) v += d[(size_t)s * stride + r];
    return v;
}

// Relu transformer.  One thread per (box, padded neuron).  With `slots` the
// bounds are first assembled from the per-column-tile sums the concretising
// contraction left (rows ordered (box, side, neuron)) and written to lb_out / ub_out.
// actL / actU (optional) receive the concrete bounds of the layer's outputs, relu(l) and
// relu(u) under a ReLU (Relu transformer, first two components), else l and u: what a
// traversal that stops on this layer is simplified against.
__global__ void relax_kernel(float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                             int out_off, int n, int ld, int batch, float *__restrict__ lamL,
                             float *__restrict__ lamU, float *__restrict__ nuU,
                             float *__restrict__ actL, float *__restrict__ actU,
                             unsigned char *__restrict__ codes, int n_relu, int relu_off,
                             const float *__restrict__ slots, int n_slots, long long slot_stride,
                             int slot_npos, int do_relax, const int *__restrict__ run_if) {
    pdl_trigger();
    pdl_wait();
    if (run_if && *run_if == 0) return;      // a re-run that is not needed (see Traversal::run_if)
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * ld) return;
    int b = (int)(idx / ld), t = (int)(idx % ld);
    float ll = 0.0f, lu = 0.0f, nu = 0.0f, al = 0.0f, au = 0.0f;
    if (t < n) {
        float l, u;
        if (slots) {
            long long rl = (2LL * b) * n + t, ru = (2LL * b + 1) * n + t;
            if (slot_npos > 0) {
                // rows ordered (box, position, side, channel): the tensor-core patch steps of a conv layer
                const int c = n / slot_npos, ch = t / slot_npos, pos = t - ch * slot_npos;
                rl = (((long long)b * slot_npos + pos) * 2) * c + ch;
                ru = rl + c;
            }
            l = slot_sum(slots, n_slots, slot_stride, rl);
            u = slot_sum(slots, n_slots, slot_stride, ru);
            CERT_ST(lb_out[(size_t)b * n_total + out_off + t], l);
            CERT_ST(ub_out[(size_t)b * n_total + out_off + t], u);
        } else {
            l = lb_out[(size_t)b * n_total + out_off + t];
            u = ub_out[(size_t)b * n_total + out_off + t];
        }
        al = l;
        au = u;
        if (do_relax) {
            al = l >= 0.0f ? l : 0.0f;
            au = u >= 0.0f ? u : 0.0f;
            bool pick_one = (__fadd_rn(l, u) >= 0.0f);   // relu_n
            ll = pick_one ? 1.0f : 0.0f;
            unsigned char code;
            if (l >= 0.0f) {                              // compute_upper, first test
                lu = 1.0f; code = 1;
            } else if (u <= 0.0f) {                       // second test
                lu = 0.0f; code = 0;
            } else {
                float den = __fsub_rn(u, l);
                lu = __fdiv_rn(u, den);
                nu = -__fdiv_rn(__fmul_rn(u, l), den);
                code = (unsigned char)(2 + (pick_one ? 1 : 0));
            }
            CERT_ST(codes[(size_t)b * n_relu + relu_off + t], code);
        }
    }
    if (actL) {
        CERT_ST(actL[idx], al);
        CERT_ST(actU[idx], au);
    }
    if (!do_relax) return;
    CERT_ST(lamL[idx], ll);
    CERT_ST(lamU[idx], lu);
    CERT_ST(nuU[idx], nu);
}

// Start of a back-substitution at a conv layer k: the expression of neuron i = (co, oy, ox) is zero except
// on the window [y0, y0+kh) x [x0, x0+kw) of every input channel, so a warp clears its row with 16-byte
// stores and then places the c_in*kh*kw window coefficients, pushed through the ReLU below as in
// relu_step_kernel (a zero coefficient contributes nothing to the row or to the constant).
__global__ void conv_expr_start_kernel(const float *__restrict__ Wk, ConvGeom gk, const float *__restrict__ bias_k,
                                       float *__restrict__ P, float *__restrict__ P_lo, float *__restrict__ d,
                                       long long rows, int n_k, int ld, int has_relu,
                                       const float *__restrict__ lamL, const float *__restrict__ lamU,
                                       const float *__restrict__ nuU, const float *__restrict__ bias_below) {
    long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (r >= rows) return;
    int b = (int)(r / (2LL * n_k));
    int upper = (int)((r / n_k) & 1);
    int i = (int)(r % n_k);
    float *prow = P + (size_t)r * ld;
    float *lrow = P_lo ? P_lo + (size_t)r * ld : nullptr;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int t = lane * 4; t < ld; t += 128) {
        CERT_ST(*reinterpret_cast<float4 *>(prow + t), zero);
        if (lrow) CERT_ST(*reinterpret_cast<float4 *>(lrow + t), zero);
    }
    __syncwarp();      // orders the clearing stores before the window stores of other lanes
    const float *ll = lamL + (size_t)b * ld, *lu = lamU + (size_t)b * ld, *nu = nuU + (size_t)b * ld;
    const int hw_o = gk.h_out * gk.w_out;
    const int co = i / hw_o;
    const int y0 = ((i / gk.w_out) % gk.h_out) * gk.stride - gk.pad;
    const int x0 = (i % gk.w_out) * gk.stride - gk.pad;
    const int khw = gk.kh * gk.kw, taps = gk.c_in * khw;
    float dacc = 0.0f;
    for (int q = lane; q < taps; q += 32) {
        const int ci = q / khw, ky = (q / gk.kw) % gk.kh, kx = q % gk.kw;
        const int iy = y0 + ky, ix = x0 + kx;
        if (iy < 0 || iy >= gk.h_in || ix < 0 || ix >= gk.w_in) continue;
        const int t = (ci * gk.h_in + iy) * gk.w_in + ix;
        const float c = Wk[(size_t)co * taps + q];
        const float qv = has_relu ? relu_backstep(c, upper, ll[t], lu[t], nu[t], dacc) : c;
        dacc = fmaf(qv, bias_below[t], dacc);
        if (lrow) {
            const float h = tf32_round(qv);
            CERT_ST(prow[t], h);
            CERT_ST(lrow[t], tf32_round(qv - h));
        } else {
            CERT_ST(prow[t], qv);
        }
    }
    dacc = warp_sum(dacc);
    if (lane == 0) CERT_ST(d[r], bias_k[i] + dacc);
}

// The same start with the columns in [y][channel][x] order (banded conv steps): the window's kh map rows are one
// contiguous piece of the row, so a warp writes the row once, 16 bytes per lane, looking up the tap of each column
// inside that piece and storing zeros elsewhere.
__global__ void conv_expr_start_ymajor_kernel(const float *__restrict__ Wk, ConvGeom gk,
                                              const float *__restrict__ bias_k, float *__restrict__ P,
                                              float *__restrict__ P_lo, float *__restrict__ d, long long rows, int n_k,
                                              int ld, int has_relu, const float *__restrict__ lamL,
                                              const float *__restrict__ lamU, const float *__restrict__ nuU,
                                              const float *__restrict__ bias_below) {
    long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (r >= rows) return;
    int b = (int)(r / (2LL * n_k));
    int upper = (int)((r / n_k) & 1);
    int i = (int)(r % n_k);
    float *prow = P + (size_t)r * ld;
    float *lrow = P_lo ? P_lo + (size_t)r * ld : nullptr;
    const float *ll = lamL + (size_t)b * ld, *lu = lamU + (size_t)b * ld, *nu = nuU + (size_t)b * ld;
    const int hw_o = gk.h_out * gk.w_out;
    const int co = i / hw_o;
    const int y0 = ((i / gk.w_out) % gk.h_out) * gk.stride - gk.pad;
    const int x0 = (i % gk.w_out) * gk.stride - gk.pad;
    const int khw = gk.kh * gk.kw, taps = gk.c_in * khw;
    const int row = gk.c_in * gk.w_in;
    const int seg_lo = max(y0, 0) * row, seg_hi = min(y0 + gk.kh, gk.h_in) * row;
    const float *wrow = Wk + (size_t)co * taps;
    float dacc = 0.0f;
    for (int t0 = lane * 4; t0 < ld; t0 += 128) {
        float hi4[4] = {0.0f, 0.0f, 0.0f, 0.0f}, lo4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (t0 + 3 >= seg_lo && t0 < seg_hi) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = t0 + e;
                if (t < seg_lo || t >= seg_hi) continue;
                const int iy = t / row, rem = t - iy * row;
                const int ci = rem / gk.w_in, ix = rem - ci * gk.w_in;
                const int kx = ix - x0;
                if (kx < 0 || kx >= gk.kw) continue;
                const float c = wrow[(ci * gk.kh + (iy - y0)) * gk.kw + kx];
                const int ts = (ci * gk.h_in + iy) * gk.w_in + ix;      // channel-major: relaxation and bias below
                const float qv = has_relu ? relu_backstep(c, upper, ll[ts], lu[ts], nu[ts], dacc) : c;
                dacc = fmaf(qv, bias_below[ts], dacc);
                if (lrow) {
                    hi4[e] = tf32_round(qv);
                    lo4[e] = tf32_round(qv - hi4[e]);
                } else {
                    hi4[e] = qv;
                }
            }
        }
        CERT_ST(*reinterpret_cast<float4 *>(prow + t0), make_float4(hi4[0], hi4[1], hi4[2], hi4[3]));
        if (lrow) CERT_ST(*reinterpret_cast<float4 *>(lrow + t0), make_float4(lo4[0], lo4[1], lo4[2], lo4[3]));
    }
    dacc = warp_sum(dacc);
    if (lane == 0) CERT_ST(d[r], bias_k[i] + dacc);
}

// Start of a back-substitution at FC layer k: row i of W_k pushed through the ReLU below, constant =
// b_k[i] + the nu terms + Q.b of the layer below.  A warp takes kStartRows consecutive neurons of one
// (box, side), 4 columns per lane, so the relaxation and bias vectors are read once for those rows.
// Q_lo != nullptr: the row is written as a TF32 pair.  With few rows (a narrow layer over a wide one) a warp
// takes one row, so that enough warps are in flight.
template <int kStartRows>
__global__ void fc_expr_start_kernel(const float *__restrict__ Wk, int ldw_k, const float *__restrict__ bias_k,
                                     float *__restrict__ Q, float *__restrict__ Q_lo, float *__restrict__ d,
                                     long long n_warps, int n_k, int n, int ld, int has_relu,
                                     const float *__restrict__ lamL, const float *__restrict__ lamU,
                                     const float *__restrict__ nuU, const float *__restrict__ bias_below, const int *__restrict__ run_if) {
    pdl_trigger();
    pdl_wait();
    if (run_if && *run_if == 0) return;      // a re-run that is not needed
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_warps) return;
    const int chunks = (n_k + kStartRows - 1) / kStartRows;
    const long long grp = w / chunks;                  // (box, side)
    const int i0 = (int)(w % chunks) * kStartRows;
    const int b = (int)(grp >> 1);
    const int upper = (int)(grp & 1);
    const long long r0 = grp * n_k + i0;
    const float *ll = lamL + (size_t)b * ld, *lu = lamU + (size_t)b * ld, *nu = nuU + (size_t)b * ld;
    float dacc[kStartRows];
#pragma unroll
    for (int rr = 0; rr < kStartRows; ++rr) dacc[rr] = 0.0f;
    for (int t = lane * 4; t < ld; t += 128) {
        const float4 bz4 = *reinterpret_cast<const float4 *>(bias_below + t);
        const float bz[4] = {bz4.x, bz4.y, bz4.z, bz4.w};
        float la[4] = {1.f, 1.f, 1.f, 1.f}, ua[4] = {1.f, 1.f, 1.f, 1.f}, na[4] = {0.f, 0.f, 0.f, 0.f};
        if (has_relu) {
            const float4 l4 = *reinterpret_cast<const float4 *>(ll + t);
            const float4 u4 = *reinterpret_cast<const float4 *>(lu + t);
            const float4 n4 = *reinterpret_cast<const float4 *>(nu + t);
            la[0] = l4.x; la[1] = l4.y; la[2] = l4.z; la[3] = l4.w;
            ua[0] = u4.x; ua[1] = u4.y; ua[2] = u4.z; ua[3] = u4.w;
            na[0] = n4.x; na[1] = n4.y; na[2] = n4.z; na[3] = n4.w;
        }
#pragma unroll
        for (int rr = 0; rr < kStartRows; ++rr) {
            if (i0 + rr >= n_k) break;
            const float4 c4 = *reinterpret_cast<const float4 *>(Wk + (size_t)(i0 + rr) * ldw_k + t);
            const float c[4] = {c4.x, c4.y, c4.z, c4.w};
            float q[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                q[e] = 0.0f;
                if (t + e < n) q[e] = has_relu ? relu_backstep(c[e], upper, la[e], ua[e], na[e], dacc[rr]) : c[e];
                dacc[rr] = fmaf(q[e], bz[e], dacc[rr]);
            }
            float *qrow = Q + (size_t)(r0 + rr) * ld + t;
            if (Q_lo) {
                float h[4], l[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    h[e] = tf32_round(q[e]);
                    l[e] = tf32_round(q[e] - h[e]);
                }
                CERT_ST(*reinterpret_cast<float4 *>(qrow), make_float4(h[0], h[1], h[2], h[3]));
                CERT_ST(*reinterpret_cast<float4 *>(Q_lo + (size_t)(r0 + rr) * ld + t), make_float4(l[0], l[1], l[2], l[3]));
            } else {
                CERT_ST(*reinterpret_cast<float4 *>(qrow), make_float4(q[0], q[1], q[2], q[3]));
            }
        }
    }
#pragma unroll
    for (int rr = 0; rr < kStartRows; ++rr) {
        const float tot = warp_sum(dacc[rr]);
        if (lane == 0 && i0 + rr < n_k) CERT_ST(d[r0 + rr], bias_k[i0 + rr] + tot);
    }
}

// ReLU back-step in place on P (expression over a layer's outputs), plus the constant's share Q.b of the
// affine step that follows; the constant comes in as a sum of slots and leaves in slot 0.

__global__ void relu_step_kernel(float *__restrict__ P,
                                 float *__restrict__ P_lo, float *__restrict__ d, int n_slots,
                                 long long slot_stride, long long rows, int n_k, int n, int ld, int has_relu,
                                 const float *__restrict__ lamL, const float *__restrict__ lamU,
                                 const float *__restrict__ nuU, const float *__restrict__ bias_below) {
    long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (r >= rows) return;
    int b = (int)(r / (2LL * n_k));
    int upper = (int)((r / n_k) & 1);
    float *prow = P + (size_t)r * ld;
    const float *ll = lamL + (size_t)b * ld, *lu = lamU + (size_t)b * ld, *nu = nuU + (size_t)b * ld;
    float dacc = 0.0f;
    // four consecutive columns per lane: 16-byte accesses (every row pitch is a multiple of 32 floats)
    for (int t = lane * 4; t < ld; t += 128) {
        float c[4], q[4];
        {
            const float4 c4 = *reinterpret_cast<const float4 *>(prow + t);
            c[0] = c4.x; c[1] = c4.y; c[2] = c4.z; c[3] = c4.w;
        }
        const float4 bz4 = *reinterpret_cast<const float4 *>(bias_below + t);
        const float bz[4] = {bz4.x, bz4.y, bz4.z, bz4.w};
        if (has_relu) {
            const float4 l4 = *reinterpret_cast<const float4 *>(ll + t);
            const float4 u4 = *reinterpret_cast<const float4 *>(lu + t);
            const float4 n4 = *reinterpret_cast<const float4 *>(nu + t);
            const float la[4] = {l4.x, l4.y, l4.z, l4.w}, ua[4] = {u4.x, u4.y, u4.z, u4.w},
                        na[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) q[e] = (t + e < n) ? relu_backstep(c[e], upper, la[e], ua[e], na[e], dacc) : 0.0f;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) q[e] = (t + e < n) ? c[e] : 0.0f;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) dacc = fmaf(q[e], bz[e], dacc);
        if (P_lo) {
            // operand form of the tensor-core contraction: q = hi + lo, both TF32
            float h[4], l[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                h[e] = tf32_round(q[e]);
                l[e] = tf32_round(q[e] - h[e]);
            }
            CERT_ST(*reinterpret_cast<float4 *>(prow + t), make_float4(h[0], h[1], h[2], h[3]));
            CERT_ST(*reinterpret_cast<float4 *>(P_lo + (size_t)r * ld + t), make_float4(l[0], l[1], l[2], l[3]));
        } else {
            CERT_ST(*reinterpret_cast<float4 *>(prow + t), make_float4(q[0], q[1], q[2], q[3]));
        }
    }
    dacc = warp_sum(dacc);
    if (lane == 0) CERT_ST(d[r], slot_sum(d, n_slots, slot_stride, r) + dacc);
}

__global__ void concretize_kernel(const float *__restrict__ P, const float *__restrict__ d, int n_slots,
                                  long long slot_stride, const float *__restrict__ l0, const float *__restrict__ u0, int n0, int ld0,
                                  long long rows, int n_k, float *__restrict__ lb_out, float *__restrict__ ub_out,
                                  int n_total, int out_off) {
    long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (r >= rows) return;
    int b = (int)(r / (2LL * n_k));
    int upper = (int)((r / n_k) & 1);
    int i = (int)(r % n_k);
    const float *prow = P + (size_t)r * ld0;
    const float *lrow = l0 + (size_t)b * ld0, *urow = u0 + (size_t)b * ld0;
    float acc = 0.0f;
    for (int s = lane; s < n0; s += 32) {
        float c = prow[s], l = lrow[s], u = urow[s];
        bool nn = (c >= 0.0f);
        acc = fmaf(c, (nn != (upper != 0)) ? l : u, acc);   // lower: c>=0 -> l ; upper: c>=0 -> u
    }
    acc = warp_sum(acc);
    if (lane == 0) {
        float v = slot_sum(d, n_slots, slot_stride, r) + acc;
        CERT_ST((upper ? ub_out : lb_out)[(size_t)b * n_total + out_off + i], v);
    }
}

inline unsigned grid_for_warps(long long warps) {
    return (unsigned)ceil_div_ll(warps, kWarpsPerBlock);
}

// Largest |x| of an array, into *out (which the caller has set to zero or an earlier maximum): the bit pattern
// of a non-negative float orders like the integer it is.
__global__ void absmax_kernel(const float *__restrict__ x, long long n, float *__restrict__ out) {
    float m = 0.0f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        m = fmaxf(m, fabsf(x[i]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<unsigned int *>(out), __float_as_uint(m));
}

}  // namespace

#ifdef CERT_BOUNDS
namespace {
__global__ void checked_store_selftest_kernel(float *p) { CERT_ST(p[0], 1.0f); }
}  // namespace
void launch_checked_store_selftest(float *p, cudaStream_t st) { checked_store_selftest_kernel<<<1, 1, 0, st>>>(p); }
#endif

void launch_absmax(const float *x, long long n, float *out, cudaStream_t st) {
    const int blocks = (int)std::min<long long>(ceil_div_ll(n, 256), 1184);
    absmax_kernel<<<blocks, 256, 0, st>>>(x, n, out);
}

// Multiprocessors of the current device (looked up once).
static int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n = v;
        else
            n = 148;
        cudaGetLastError();
    }
    return n;
}

bool pdl_enabled() {
    static const bool on = [] {
        const char *e = std::getenv("CERT_PDL");
        return !(e && e[0] == '0');
    }();
    return on;
}

void launch_box(const float *centers, float eps, float lo, float hi, int batch, int n0, int ld0, float *l0,
                float *u0, cudaStream_t st) {
    long long n = (long long)batch * ld0;
    launch_chained(box_kernel, dim3((unsigned)ceil_div_ll(n, 256)), dim3(256), 0, st, centers, eps, lo, hi, batch, n0, ld0,
                   l0, u0);
}

void launch_first_layer_bounds(const LayerDev &L, const float *l0, const float *u0, int ld0, int batch,
                               float *lb_out, float *ub_out, int n_total, cudaStream_t st) {
    long long warps = (long long)batch * L.n_out;
    if (L.kind == CERT_LAYER_CONV2D) {
        launch_chained(first_layer_conv_kernel, dim3((unsigned)ceil_div_ll(warps, 128)), dim3(128), 0, st, L.W, L.bias_n,
                       geom_of(L), L.n_out, l0, u0, ld0, batch, lb_out, ub_out, n_total, L.out_off);
        return;
    }
    // two neurons per warp: the box row is read once for both (measured best of 1, 2, 4, 8 on the 1024-wide layers)
    constexpr int kPerWarp = 2;
    const long long fc_warps = (long long)batch * ((L.n_out + kPerWarp - 1) / kPerWarp);
    const bool vec_ok = L.ld_in % 4 == 0 && ld0 % 4 == 0 && 4 * ((L.n_in + 3) / 4) <= L.ld_in &&
                        4 * ((L.n_in + 3) / 4) <= ld0 && (reinterpret_cast<uintptr_t>(L.W) & 15) == 0 &&
                        (reinterpret_cast<uintptr_t>(l0) & 15) == 0 && (reinterpret_cast<uintptr_t>(u0) & 15) == 0;
    if (vec_ok)
        launch_chained(first_layer_vec_kernel<kPerWarp>, dim3(grid_for_warps(fc_warps)), dim3(kWarpsPerBlock * 32), 0,
                       st, L.W, L.bias_n, L.n_in, L.ld_in, L.n_out, l0, u0, ld0, batch, lb_out, ub_out, n_total,
                       L.out_off);
    else
        launch_chained(first_layer_kernel<kPerWarp>, dim3(grid_for_warps(fc_warps)), dim3(kWarpsPerBlock * 32), 0, st,
                       L.W, L.bias_n, L.n_in, L.ld_in, L.n_out, l0, u0, ld0, batch, lb_out, ub_out, n_total, L.out_off);
}

void launch_relax(const LayerDev &L, float *lb_out, float *ub_out, int n_total, int batch,
                  unsigned char *codes, int n_relu, const float *slots, int n_slots, long long slot_stride,
                  cudaStream_t st, int slot_npos, const int *run_if) {
    long long n = (long long)batch * L.ld_out;
    launch_chained(relax_kernel, dim3((unsigned)ceil_div_ll(n, 256)), dim3(256), 0, st, lb_out, ub_out, n_total,
                   L.out_off, L.n_out, L.ld_out, batch, L.lamL, L.lamU, L.nuU, L.actL, L.actU, codes, n_relu, L.relu_off,
                   slots, n_slots, slot_stride, slot_npos, L.relu_after, run_if);
}

void launch_init_expr(const LayerDev &Lk, const LayerDev &Lb, int batch, float *Q, float *Q_lo, float *d,
                      cudaStream_t st, int y_major, const int *run_if) {
    long long rows = 2LL * batch * Lk.n_out;
    if (Lk.kind != CERT_LAYER_FC && y_major) {
        conv_expr_start_ymajor_kernel<<<grid_for_warps(rows), kWarpsPerBlock * 32, 0, st>>>(
            Lk.W, geom_of(Lk), Lk.bias_n, Q, Q_lo, d, rows, Lk.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL, Lb.lamU,
            Lb.nuU, Lb.bias_n);
        return;
    }
    if (Lk.kind != CERT_LAYER_FC) {
        conv_expr_start_kernel<<<grid_for_warps(rows), kWarpsPerBlock * 32, 0, st>>>(
            Lk.W, geom_of(Lk), Lk.bias_n, Q, Q_lo, d, rows, Lk.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL, Lb.lamU,
            Lb.nuU, Lb.bias_n);
        return;
    }
    const long long warps4 = 2LL * batch * ((Lk.n_out + 3) / 4);
    if (warps4 >= 32LL * sm_count()) {          // enough four-row warps to fill the multiprocessors
        launch_chained(fc_expr_start_kernel<4>, dim3(grid_for_warps(warps4)), dim3(kWarpsPerBlock * 32), 0, st, Lk.W,
                       Lk.ld_in, Lk.bias_n, Q, Q_lo, d, warps4, Lk.n_out, Lb.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL,
                       Lb.lamU, Lb.nuU, Lb.bias_n, run_if);
    } else {
        launch_chained(fc_expr_start_kernel<1>, dim3(grid_for_warps(rows)), dim3(kWarpsPerBlock * 32), 0, st, Lk.W,
                       Lk.ld_in, Lk.bias_n, Q, Q_lo, d, rows, Lk.n_out, Lb.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL,
                       Lb.lamU, Lb.nuU, Lb.bias_n, run_if);
    }
}

void launch_relu_step(const LayerDev &Lj, int batch, int n_k, float *P, float *P_lo, float *d, int n_slots,
                      long long slot_stride, cudaStream_t st) {
    long long rows = 2LL * batch * n_k;
    relu_step_kernel<<<grid_for_warps(rows), kWarpsPerBlock * 32, 0, st>>>(
        P, P_lo, d, n_slots, slot_stride, rows, n_k, Lj.n_out, Lj.ld_out, Lj.relu_after, Lj.lamL,
        Lj.lamU, Lj.nuU, Lj.bias_n);
}

void launch_add_skip(float *P, const float *S_hi, const float *S_lo, int identity, long long rows, int n, int ld,
                     int n_k, cudaStream_t st) {
    const long long total = rows * (long long)ld;
    add_skip_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(P, S_hi, S_lo, identity, total, n, ld, n_k);
}

void launch_add_act_bounds(const LayerDev &Lk, const LayerDev &Ls, int batch, float *lb_out, float *ub_out,
                           int n_total, cudaStream_t st) {
    const long long n = (long long)batch * Lk.n_out;
    add_act_bounds_kernel<<<(unsigned)ceil_div_ll(n, 256), 256, 0, st>>>(lb_out, ub_out, n_total, Lk.out_off, Lk.n_out,
                                                                       batch, Ls.actL, Ls.actU, Ls.ld_out);
}

void launch_skip_concretize(const float *S_hi, const float *S_lo, int identity, const LayerDev &Ls, long long rows,
                            const LayerDev &Lk, float *slot, float *lb_out, float *ub_out, int n_total,
                            cudaStream_t st) {
    skip_concretize_kernel<<<grid_for_warps(rows), kWarpsPerBlock * 32, 0, st>>>(
        S_hi, S_lo, identity, Ls.actL, Ls.actU, Ls.ld_out, rows, Ls.n_out, Ls.ld_out, Lk.n_out, slot, lb_out, ub_out,
        n_total, Lk.out_off);
}

void launch_concretize(const float *P, const float *d, int n_slots, long long slot_stride, const float *l0,
                       const float *u0, int n0, int ld0, int batch, int n_k, float *lb_out, float *ub_out, int n_total, int out_off,
                       cudaStream_t st) {
    long long rows = 2LL * batch * n_k;
    concretize_kernel<<<grid_for_warps(rows), kWarpsPerBlock * 32, 0, st>>>(P, d, n_slots, slot_stride, l0, u0, n0, ld0, rows, n_k,
                                                                          lb_out, ub_out, n_total, out_off);
}

}  // namespace cert
