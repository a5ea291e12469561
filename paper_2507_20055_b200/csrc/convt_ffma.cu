// Conv back-step: a row's coefficient map over the outputs of a conv layer is
// pushed through the layer by the exact transpose of the convolution
// (Appendix B: a dense block times a convolution block is conv_transpose2d):
//
//   P[r][ci][iy][ix] = sum over (co, ky, kx) with (iy + pad - ky) = stride * oy and
//                      (ix + pad - kx) = stride * ox of  Q[r][co][oy][ox] * W[co][ci][ky][kx]
//
// and what follows the step on the path is applied to P while it is still in
// registers: either the ReLU back-step through the layer below
// (replace_lower/upper, clamp form of Section 4.3) plus the constant's share
// P'.b of the next affine step, or the concretisation against the input box
// (map(simplify_lower/upper)), in which case P is never stored.
//
// Implicit GEMM on the fp32 FMA units (the channel count below a conv layer is
// 3..16: too narrow an N for the tensor cores).  Input pixels fall into
// stride x stride classes by ((iy + pad) mod stride, (ix + pad) mod stride);
// every pixel of a class uses the same kernel taps, so a warp that works on one
// class reads its weights as warp-uniform 16-byte shared-memory loads.  A block
// stages the maps of RB rows in shared memory inside a zero halo (no bounds
// tests in the inner loop); a thread accumulates PXT pixels x CT channels in
// registers.  A lane always works for the same row of the group (lane / (32/RB)),
// so a row's constant is summed in registers, then across the lanes of its
// group by shuffles and across warps in a fixed order: no atomics.
//
// Stride 2 with at most 4 channels below (an image layer): the four classes of the pixels
// (2uy + cy - pad, 2ux + cx - pad) read the same coefficients Q[co][uy - dy][ux - dx], so a thread
// takes all four classes of its positions (uy, ux) at once and every coefficient read from shared
// memory feeds 4 x CT FMAs instead of CT (convt_s2_kernel).
#include "common.cuh"

namespace cert {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxStride = 4;
constexpr int kMaxRowsPerGroup = 8;
constexpr size_t kSmemBudget = 100 * 1024;   // two blocks per multiprocessor: one stages while the other computes

// Shared-memory plan of one conv layer's back-step, derived on the host.
struct ConvtPlan {
    int halo_y, halo_x;      // zero rows / columns before the map
    int HP, WP;              // padded map height / width
    int map_stride;          // floats between consecutive rows' staged maps
    int cpad;                // c_in rounded up to 4 (weights are staged as [co][ky][kx][cpad])
    int rows_per_group;      // rows staged per pass: a power of two <= 8
    size_t smem_bytes;
    // stride-2 form: taps per axis (ceil(k/2)), extent of the position grid; n_w = staged weight count
    int s2;                  // 1: convt_s2_kernel applies
    int ty, tx, hu, wu, n_w;
};

struct AxisRange { int lo, hi; };

// Range of o = (i + pad - k) / stride over the input pixels and taps that divide evenly.
AxisRange output_range(int n_in, int k, int stride, int pad) {
    AxisRange r{0, -1};
    bool first = true;
    for (int i = 0; i < n_in; ++i)
        for (int t = 0; t < k; ++t) {
            int v = i + pad - t;
            if (v % stride != 0) continue;          // the remainder keeps the sign, so this holds for v < 0 too
            int o = v / stride;
            if (first) { r.lo = r.hi = o; first = false; }
            r.lo = std::min(r.lo, o);
            r.hi = std::max(r.hi, o);
        }
    return r;
}

ConvtPlan make_plan(const LayerDev &L) {
    ConvtPlan p{};
    AxisRange ry = output_range(L.h_in, L.kh, L.stride, L.pad);
    AxisRange rx = output_range(L.w_in, L.kw, L.stride, L.pad);
    p.halo_y = ry.lo < 0 ? -ry.lo : 0;
    p.halo_x = rx.lo < 0 ? -rx.lo : 0;
    p.HP = p.halo_y + std::max(L.h_out, ry.hi + 1);
    p.WP = p.halo_x + std::max(L.w_out, rx.hi + 1);
    p.cpad = round_up(L.c_in, 4);
    p.n_w = L.c_out * L.kh * L.kw * p.cpad;
    // Stride-2 form: positions u in [0, hu) x [0, wu) cover every class's pixels (u = (i + pad - c) / 2);
    // taps dy < ty, dx < tx; weights staged with the kernel padded to 2*ty x 2*tx (zeros), and a halo of
    // at least ty-1, tx-1 so that a position whose tap does not exist reads staged zeros or staged data,
    // never anything else.
    p.ty = (L.kh + 1) / 2;
    p.tx = (L.kw + 1) / 2;
    p.s2 = (L.stride == 2 && L.c_in <= 4 && p.ty == p.tx && p.ty >= 1 && p.ty <= 3) ? 1 : 0;
    if (p.s2) {
        p.hu = (L.h_in - 1 + L.pad) / 2 + 1;
        p.wu = (L.w_in - 1 + L.pad) / 2 + 1;
        p.halo_y = std::max(p.halo_y, p.ty - 1);
        p.halo_x = std::max(p.halo_x, p.tx - 1);
        p.HP = p.halo_y + std::max(std::max(L.h_out, ry.hi + 1), p.hu);
        p.WP = p.halo_x + std::max(std::max(L.w_out, rx.hi + 1), p.wu);
        p.n_w = L.c_out * (2 * p.ty) * (2 * p.tx) * p.cpad;
    }
    const size_t w_bytes = sizeof(float) * (size_t)p.n_w;
    const size_t fixed = w_bytes + sizeof(float) * kWarps * kMaxRowsPerGroup;
    const int map = L.c_out * p.HP * p.WP;
    p.rows_per_group = 0;
    for (int rb = kMaxRowsPerGroup; rb >= 1; rb /= 2) {
        // The 32/rb lanes that work for one row read consecutive pixels; a map stride congruent to
        // 32/rb modulo 32 puts the rows' lane groups on distinct banks.
        int ms = map;
        while (ms % 32 != (32 / rb) % 32) ++ms;
        size_t bytes = fixed + sizeof(float) * (size_t)ms * rb;
        if (bytes <= kSmemBudget) {
            p.rows_per_group = rb;
            p.map_stride = ms;
            p.smem_bytes = bytes;
            break;
        }
    }
    return p;
}

// Coefficient of a residual connection that ends on the neurons this step reaches (0 without one).
__device__ __forceinline__ float skip_addend(const ConvtEpilogue &ep, long long r, int t, int ld_in) {
    float s = 0.0f;
    if (ep.add_hi) {
        const size_t o = (size_t)r * ld_in + t;
        s = ep.add_hi[o];
        if (ep.add_lo) s += ep.add_lo[o];
    }
    if (ep.add_identity && t == (int)(r % ep.n_k)) s += 1.0f;
    return s;
}

__device__ __forceinline__ float tf32_round(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

__device__ __forceinline__ void cp_async4(float *smem_dst, const float *gsrc, bool live) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    const int src_bytes = live ? 4 : 0;     // 0: nothing is read, the word is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(gsrc), "r"(src_bytes) : "memory");
}

// acc[i][c] += sum over output channels and the class's taps of Q * W for PXT pixels x CT channels.
// q[i]: this lane's pixels in the staged maps (tap (0,0), channel 0); w: the class's tap (0,0) of
// output channel 0 at input channel c0.  TY, TX: taps per axis when known at compile time (the loops
// then unroll and the tap offsets live in registers), 0 = take n_my, n_mx at run time.
template <int CT, int PXT, int TY, int TX>
__device__ __forceinline__ void accumulate_taps(float (&acc)[PXT][CT], const float *const (&q)[PXT],
                                                const float *w, int c_out, int plane, int w_co_stride,
                                                int w_my_stride, int w_mx_stride, int WP, int n_my, int n_mx) {
    constexpr int CTL = (CT + 3) / 4 * 4;       // weights are read in 16-byte pieces
    const int ty = TY > 0 ? TY : n_my, tx = TX > 0 ? TX : n_mx;
#pragma unroll 2
    for (int co = 0; co < c_out; ++co) {
        const float *wc = w + co * w_co_stride;
        const int qc = co * plane;
#pragma unroll
        for (int my = 0; my < ty; ++my) {
#pragma unroll
            for (int mx = 0; mx < tx; ++mx) {
                float wv[CTL];
#pragma unroll
                for (int c4 = 0; c4 < CTL; c4 += 4) {
                    const float4 w4 = *reinterpret_cast<const float4 *>(wc + my * w_my_stride + mx * w_mx_stride + c4);
                    wv[c4] = w4.x; wv[c4 + 1] = w4.y; wv[c4 + 2] = w4.z; wv[c4 + 3] = w4.w;
                }
                const int shift = qc - my * WP - mx;
#pragma unroll
                for (int i = 0; i < PXT; ++i) {
                    const float qv = q[i][shift];
#pragma unroll
                    for (int c = 0; c < CT; ++c) acc[i][c] = fmaf(qv, wv[c], acc[i][c]);
                }
            }
        }
    }
}

// The same for a channel chunk of which only `left` (< round_up(CT, 4)) channels exist in the staged rows.
template <int CT, int PXT>
__device__ __forceinline__ void accumulate_tail(float (&acc)[PXT][CT], const float *const (&q)[PXT],
                                                const float *w, int c_out, int plane, int w_co_stride,
                                                int w_my_stride, int w_mx_stride, int WP, int n_my, int n_mx,
                                                int left) {
    for (int co = 0; co < c_out; ++co) {
        for (int my = 0; my < n_my; ++my) {
            for (int mx = 0; mx < n_mx; ++mx) {
                const float *wc = w + co * w_co_stride + my * w_my_stride + mx * w_mx_stride;
                float wv[CT];
#pragma unroll
                for (int c = 0; c < CT; ++c) wv[c] = c < left ? wc[c] : 0.0f;
                const int shift = co * plane - my * WP - mx;
#pragma unroll
                for (int i = 0; i < PXT; ++i) {
                    const float qv = q[i][shift];
#pragma unroll
                    for (int c = 0; c < CT; ++c) acc[i][c] = fmaf(qv, wv[c], acc[i][c]);
                }
            }
        }
    }
}

// Q [rows][ld_out] maps (c_out, h_out, w_out); the result maps (c_in, h_in, w_in) with pitch ld_in.
// Wct: weights laid out [c_out][kh][kw][c_in].
template <int CT, int PXT, int EPI>
__global__ void __launch_bounds__(kThreads, 2)
convt_kernel(const float *__restrict__ Q, int ld_out, int ld_in, const float *__restrict__ Wct, ConvGeom g,
             ConvtPlan pl, long long rows, ConvtEpilogue ep) {
    extern __shared__ __align__(16) float smem[];
    const int n_out = g.c_out * g.h_out * g.w_out;
    const int n_in = g.c_in * g.h_in * g.w_in;
    const int hw_in = g.h_in * g.w_in, hw_out = g.h_out * g.w_out;
    const int n_w = g.c_out * g.kh * g.kw * pl.cpad;
    const int RB = pl.rows_per_group;
    const int G = 32 / RB;             // lanes per row of the group
    const int plane = pl.HP * pl.WP;
    float *Ws = smem;                  // [c_out][kh][kw][cpad]
    float *red = smem + pl.n_w;        // [kWarps][kMaxRowsPerGroup] partial row constants
    float *Qs = red + kWarps * kMaxRowsPerGroup;   // [RB][map_stride], each map [c_out][HP][WP] inside its halo
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rl = lane / G, gl = lane % G;

    for (int i = threadIdx.x; i < n_w; i += kThreads) {
        int ci = i % pl.cpad, tap = i / pl.cpad;
        Ws[i] = ci < g.c_in ? Wct[(size_t)tap * g.c_in + ci] : 0.0f;
    }
    for (int i = threadIdx.x; i < RB * pl.map_stride; i += kThreads) Qs[i] = 0.0f;   // halos stay zero

    const int s = g.stride;
    const int n_classes = s * s;
    const int d_ox = kThreads % g.w_out, d_oy = (kThreads / g.w_out) % g.h_out, d_co = kThreads / hw_out;

    for (long long r0 = (long long)blockIdx.x * RB; r0 < rows; r0 += (long long)gridDim.x * RB) {
        __syncthreads();
        // Stage the maps of rows r0 .. r0+RB-1 with asynchronous 4-byte copies (rows past the end are
        // zero-filled).  The element index advances by the block size, its (co, oy, ox) split with it.
        for (int q = 0; q < RB; ++q) {
            const bool live = r0 + q < rows;
            const float *qrow = Q + (size_t)(live ? r0 + q : r0) * ld_out;
            float *qs = Qs + q * pl.map_stride + pl.halo_y * pl.WP + pl.halo_x;
            int e = threadIdx.x;
            int co = e / hw_out, oy = (e % hw_out) / g.w_out, ox = e % g.w_out;
            for (; e < n_out; e += kThreads) {
                cp_async4(qs + co * plane + oy * pl.WP + ox, qrow + e, live);
                ox += d_ox;
                if (ox >= g.w_out) { ox -= g.w_out; ++oy; }
                oy += d_oy;
                if (oy >= g.h_out) { oy -= g.h_out; ++co; }
                co += d_co;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();

        // This lane's row, and where its relaxation / box vectors start.
        const long long r = r0 + rl;
        const bool row_ok = r < rows;
        const long long rr = row_ok ? r : 0;
        const int box = (int)(rr / (2LL * ep.n_k));
        const int upper = (int)((rr / ep.n_k) & 1);
        const size_t vec = (size_t)box * ld_in;
        float dacc = 0.0f;

        // Work units: (class, chunk of G*PXT pixels); every lane group of the warp does the chunk for its row.
        int unit_base = 0;
        for (int cls = 0; cls < n_classes; ++cls) {
            const int cy = cls / s, cx = cls % s;
            // pixels of the class: iy = cy - pad + s*uy, 0 <= iy < h_in; then oy = uy - my for ky = cy + s*my
            const int uy0 = (g.pad - cy + s - 1) / s, ux0 = (g.pad - cx + s - 1) / s;   // numerators are >= 0
            const int uy1 = (g.h_in - 1 + g.pad - cy >= 0) ? (g.h_in - 1 + g.pad - cy) / s : -1;
            const int ux1 = (g.w_in - 1 + g.pad - cx >= 0) ? (g.w_in - 1 + g.pad - cx) / s : -1;
            const int Hc = uy1 - uy0 + 1, Wc = ux1 - ux0 + 1;
            const int n_my = cy < g.kh ? (g.kh - cy + s - 1) / s : 0;
            const int n_mx = cx < g.kw ? (g.kw - cx + s - 1) / s : 0;
            if (Hc <= 0 || Wc <= 0) continue;
            const int pixels = Hc * Wc;
            const int units = (pixels + G * PXT - 1) / (G * PXT);
            const int first = ((warp - unit_base) % kWarps + kWarps) % kWarps;   // units go round the warps
            for (int u = first; u < units; u += kWarps) {
                int q_off[PXT], p_off[PXT];
                bool ok[PXT];
#pragma unroll
                for (int i = 0; i < PXT; ++i) {
                    const int p = u * (G * PXT) + i * G + gl;
                    ok[i] = p < pixels;
                    const int pc = ok[i] ? p : 0;
                    const int uy = pc / Wc, ux = pc % Wc;
                    q_off[i] = rl * pl.map_stride + (uy0 + uy + pl.halo_y) * pl.WP + (ux0 + ux + pl.halo_x);
                    p_off[i] = (cy - g.pad + s * (uy0 + uy)) * g.w_in + (cx - g.pad + s * (ux0 + ux));
                    ok[i] = ok[i] && row_ok;
                }
                for (int c0 = 0; c0 < g.c_in; c0 += CT) {
                    float acc[PXT][CT];
#pragma unroll
                    for (int i = 0; i < PXT; ++i)
#pragma unroll
                        for (int c = 0; c < CT; ++c) acc[i][c] = 0.0f;
                    {
                        const float *qp[PXT];
#pragma unroll
                        for (int i = 0; i < PXT; ++i) qp[i] = Qs + q_off[i];
                        // weights of the class's first tap (ky, kx) = (cy, cx); further taps are s apart.
                        // A channel chunk that starts past the padded channel count cannot occur (c0 < c_in <= cpad);
                        // a chunk wider than what is left reads the zero padding up to a multiple of 4 only.
                        const float *w0 = Ws + (cy * g.kw + cx) * pl.cpad + c0;
                        const int w_co = g.kh * g.kw * pl.cpad, w_my = s * g.kw * pl.cpad, w_mx = s * pl.cpad;
                        const bool whole = c0 + ((CT + 3) / 4 * 4) <= pl.cpad;   // the 16-byte reads stay inside the channel row
                        if (!whole) {
                            accumulate_tail<CT, PXT>(acc, qp, w0, g.c_out, plane, w_co, w_my, w_mx, pl.WP, n_my, n_mx,
                                                     pl.cpad - c0);
                        } else if (n_my == 2 && n_mx == 2) {
                            accumulate_taps<CT, PXT, 2, 2>(acc, qp, w0, g.c_out, plane, w_co, w_my, w_mx, pl.WP, 2, 2);
                        } else if (n_my == 1 && n_mx == 1) {
                            accumulate_taps<CT, PXT, 1, 1>(acc, qp, w0, g.c_out, plane, w_co, w_my, w_mx, pl.WP, 1, 1);
                        } else if (n_my == 3 && n_mx == 3) {
                            accumulate_taps<CT, PXT, 3, 3>(acc, qp, w0, g.c_out, plane, w_co, w_my, w_mx, pl.WP, 3, 3);
                        } else {
                            accumulate_taps<CT, PXT, 0, 0>(acc, qp, w0, g.c_out, plane, w_co, w_my, w_mx, pl.WP, n_my, n_mx);
                        }
                    }
                    // ---- what follows the step on the path, per element ----
#pragma unroll
                    for (int i = 0; i < PXT; ++i) {
                        if (!ok[i]) continue;
#pragma unroll
                        for (int c = 0; c < CT; ++c) {
                            if (c0 + c >= g.c_in) continue;
                            const int t = (c0 + c) * hw_in + p_off[i];
                            const float v = acc[i][c] + (EPI == CONVT_EPI_RELU ? skip_addend(ep, r, t, ld_in) : 0.0f);
                            const bool nonneg = (v >= 0.0f);
                            if (EPI == CONVT_EPI_CONCRETIZE) {
                                // lower rows: c >= 0 ? c*l : c*u; upper rows: c >= 0 ? c*u : c*l
                                const float bnd = (nonneg != (upper != 0)) ? ep.l0[vec + t] : ep.u0[vec + t];
                                dacc = fmaf(v, bnd, dacc);
                            } else {
                                float qv = v;
                                if (ep.has_relu) {
                                    const bool use_lower = upper ? !nonneg : nonneg;
                                    if (use_lower) {
                                        qv = v * ep.lamL[vec + t];
                                    } else {
                                        dacc = fmaf(v, ep.nuU[vec + t], dacc);
                                        qv = v * ep.lamU[vec + t];
                                    }
                                }
                                dacc = fmaf(qv, ep.bias_below[t], dacc);
                                const size_t o = (size_t)r * ld_in + t;
                                if (ep.P_lo) {
                                    const float h = tf32_round(qv);
                                    CERT_ST(ep.P[o], h);
                                    CERT_ST(ep.P_lo[o], tf32_round(qv - h));
                                } else {
                                    CERT_ST(ep.P[o], qv);
                                }
                            }
                        }
                    }
                }
            }
            unit_base += units;
        }

        // Row constants: lanes of a group by shuffles, warps in warp order.
        for (int o = 1; o < G; o <<= 1) dacc += __shfl_xor_sync(0xffffffffu, dacc, o);
        if (gl == 0) red[warp * kMaxRowsPerGroup + rl] = dacc;
        __syncthreads();
        if (threadIdx.x < RB && r0 + threadIdx.x < rows) {
            const long long row = r0 + threadIdx.x;
            float tot = ep.d_in[row];
            for (int sl = 1; sl < ep.n_slots_in; ++sl) tot += ep.d_in[(size_t)sl * ep.slot_stride + row];
            for (int w2 = 0; w2 < kWarps; ++w2) tot += red[w2 * kMaxRowsPerGroup + threadIdx.x];
            if (EPI == CONVT_EPI_CONCRETIZE) {
                const int b2 = (int)(row / (2LL * ep.n_k)), up2 = (int)((row / ep.n_k) & 1), i2 = (int)(row % ep.n_k);
                CERT_ST((up2 ? ep.ub_out : ep.lb_out)[(size_t)b2 * ep.n_total + ep.out_off + i2], tot);
            } else {
                CERT_ST(ep.d_out[row], tot);
            }
        }
        if (EPI == CONVT_EPI_RELU) {
            // keep the padded tail of the rows at zero
            for (int q = 0; q < RB; ++q) {
                if (r0 + q >= rows) break;
                const size_t o = (size_t)(r0 + q) * ld_in;
                for (int t = n_in + threadIdx.x; t < ld_in; t += kThreads) {
                    CERT_ST(ep.P[o + t], 0.0f);
                    if (ep.P_lo) CERT_ST(ep.P_lo[o + t], 0.0f);
                }
            }
        }
    }
}

// One element v = P[r][t] of the back-step's result: ReLU back-step through the layer below and the
// constant's share of the next affine step (result stored), or its term of the concretisation.
template <int EPI>
__device__ __forceinline__ void finish_element(float v, int t, long long r, int upper, size_t vec, int ld_in,
                                               const ConvtEpilogue &ep, float &dacc) {
    if (EPI == CONVT_EPI_RELU) v += skip_addend(ep, r, t, ld_in);
    const bool nonneg = (v >= 0.0f);
    if (EPI == CONVT_EPI_CONCRETIZE) {
        // lower rows: c >= 0 ? c*l : c*u; upper rows: c >= 0 ? c*u : c*l
        const float bnd = (nonneg != (upper != 0)) ? ep.l0[vec + t] : ep.u0[vec + t];
        dacc = fmaf(v, bnd, dacc);
    } else {
        float qv = v;
        if (ep.has_relu) {
            const bool use_lower = upper ? !nonneg : nonneg;
            if (use_lower) {
                qv = v * ep.lamL[vec + t];
            } else {
                dacc = fmaf(v, ep.nuU[vec + t], dacc);
                qv = v * ep.lamU[vec + t];
            }
        }
        dacc = fmaf(qv, ep.bias_below[t], dacc);
        const size_t o = (size_t)r * ld_in + t;
        if (ep.P_lo) {
            const float h = tf32_round(qv);
            CERT_ST(ep.P[o], h);
            CERT_ST(ep.P_lo[o], tf32_round(qv - h));
        } else {
            CERT_ST(ep.P[o], qv);
        }
    }
}

// Stride 2, c_in <= 4.  A thread takes PXT positions (uy, ux) of its row and, for each, the four
// pixels (2uy + cy - pad, 2ux + cx - pad), cy, cx in {0, 1}; tap (dy, dx) of class (cy, cx) is kernel
// element (cy + 2dy, cx + 2dx) and reads Q[co][uy - dy][ux - dx] for every class.  Weights are staged
// as [c_out][2*T][2*T][cpad] with zeros where the kernel has no such element.
template <int CT, int PXT, int T, int EPI>
__global__ void __launch_bounds__(kThreads, 2)
convt_s2_kernel(const float *__restrict__ Q, int ld_out, int ld_in, const float *__restrict__ Wct, ConvGeom g,
                ConvtPlan pl, long long rows, ConvtEpilogue ep) {
    extern __shared__ __align__(16) float smem[];
    const int n_out = g.c_out * g.h_out * g.w_out;
    const int n_in = g.c_in * g.h_in * g.w_in;
    const int hw_in = g.h_in * g.w_in, hw_out = g.h_out * g.w_out;
    const int RB = pl.rows_per_group;
    const int G = 32 / RB;             // lanes per row of the group
    const int plane = pl.HP * pl.WP;
    float *Ws = smem;                  // [c_out][2T][2T][cpad]
    float *red = smem + pl.n_w;        // [kWarps][kMaxRowsPerGroup] partial row constants
    float *Qs = red + kWarps * kMaxRowsPerGroup;   // [RB][map_stride], each map [c_out][HP][WP] inside its halo
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rl = lane / G, gl = lane % G;

    for (int i = threadIdx.x; i < pl.n_w; i += kThreads) {
        const int ci = i % pl.cpad;
        int rest = i / pl.cpad;
        const int kx = rest % (2 * T); rest /= 2 * T;
        const int ky = rest % (2 * T);
        const int co = rest / (2 * T);
        const bool real = ci < g.c_in && ky < g.kh && kx < g.kw;
        Ws[i] = real ? Wct[(((size_t)co * g.kh + ky) * g.kw + kx) * g.c_in + ci] : 0.0f;
    }
    for (int i = threadIdx.x; i < RB * pl.map_stride; i += kThreads) Qs[i] = 0.0f;   // halos stay zero

    const int d_ox = kThreads % g.w_out, d_oy = (kThreads / g.w_out) % g.h_out, d_co = kThreads / hw_out;
    const int positions = pl.hu * pl.wu;
    const int units = (positions + G * PXT - 1) / (G * PXT);
    const int w_co = 4 * T * T * pl.cpad, w_ky = 2 * T * pl.cpad;

    for (long long r0 = (long long)blockIdx.x * RB; r0 < rows; r0 += (long long)gridDim.x * RB) {
        __syncthreads();
        for (int q = 0; q < RB; ++q) {
            const bool live = r0 + q < rows;
            const float *qrow = Q + (size_t)(live ? r0 + q : r0) * ld_out;
            float *qs = Qs + q * pl.map_stride + pl.halo_y * pl.WP + pl.halo_x;
            int e = threadIdx.x;
            int co = e / hw_out, oy = (e % hw_out) / g.w_out, ox = e % g.w_out;
            for (; e < n_out; e += kThreads) {
                cp_async4(qs + co * plane + oy * pl.WP + ox, qrow + e, live);
                ox += d_ox;
                if (ox >= g.w_out) { ox -= g.w_out; ++oy; }
                oy += d_oy;
                if (oy >= g.h_out) { oy -= g.h_out; ++co; }
                co += d_co;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();

        const long long r = r0 + rl;
        const bool row_ok = r < rows;
        const long long rr = row_ok ? r : 0;
        const int box = (int)(rr / (2LL * ep.n_k));
        const int upper = (int)((rr / ep.n_k) & 1);
        const size_t vec = (size_t)box * ld_in;
        float dacc = 0.0f;
        for (int u = warp; u < units; u += kWarps) {
            int q_off[PXT], uy[PXT], ux[PXT];
            bool ok[PXT];
#pragma unroll
            for (int i = 0; i < PXT; ++i) {
                const int p = u * (G * PXT) + i * G + gl;
                ok[i] = p < positions && row_ok;
                const int pc = p < positions ? p : 0;
                uy[i] = pc / pl.wu;
                ux[i] = pc % pl.wu;
                q_off[i] = rl * pl.map_stride + (uy[i] + pl.halo_y) * pl.WP + (ux[i] + pl.halo_x);
            }
            float acc[PXT][4][CT];
#pragma unroll
            for (int i = 0; i < PXT; ++i)
#pragma unroll
                for (int cls = 0; cls < 4; ++cls)
#pragma unroll
                    for (int c = 0; c < CT; ++c) acc[i][cls][c] = 0.0f;
#pragma unroll 2
            for (int co = 0; co < g.c_out; ++co) {
                const float *wc = Ws + co * w_co;
                const float *qc = Qs + co * plane;
#pragma unroll
                for (int dy = 0; dy < T; ++dy) {
#pragma unroll
                    for (int dx = 0; dx < T; ++dx) {
                        float qv[PXT];
#pragma unroll
                        for (int i = 0; i < PXT; ++i) qv[i] = qc[q_off[i] - dy * pl.WP - dx];
#pragma unroll
                        for (int cy = 0; cy < 2; ++cy) {
#pragma unroll
                            for (int cx = 0; cx < 2; ++cx) {
                                // kernel element (cy + 2dy, cx + 2dx), channels 0..3 (cpad = 4 here)
                                const float4 w4 = *reinterpret_cast<const float4 *>(
                                    wc + (cy + 2 * dy) * w_ky + (cx + 2 * dx) * pl.cpad);
                                const float wv[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                                for (int i = 0; i < PXT; ++i)
#pragma unroll
                                    for (int c = 0; c < CT; ++c)
                                        acc[i][cy * 2 + cx][c] = fmaf(qv[i], wv[c], acc[i][cy * 2 + cx][c]);
                            }
                        }
                    }
                }
            }
            // ---- what follows the step on the path, per element ----
#pragma unroll
            for (int i = 0; i < PXT; ++i) {
                if (!ok[i]) continue;
#pragma unroll
                for (int cy = 0; cy < 2; ++cy) {
                    const int iy = 2 * uy[i] + cy - g.pad;
                    if (iy < 0 || iy >= g.h_in) continue;
#pragma unroll
                    for (int cx = 0; cx < 2; ++cx) {
                        const int ix = 2 * ux[i] + cx - g.pad;
                        if (ix < 0 || ix >= g.w_in) continue;
#pragma unroll
                        for (int c = 0; c < CT; ++c) {
                            if (c >= g.c_in) continue;
                            finish_element<EPI>(acc[i][cy * 2 + cx][c], c * hw_in + iy * g.w_in + ix, r, upper, vec,
                                                ld_in, ep, dacc);
                        }
                    }
                }
            }
        }
        // Row constants: lanes of a group by shuffles, warps in warp order.
        for (int o = 1; o < G; o <<= 1) dacc += __shfl_xor_sync(0xffffffffu, dacc, o);
        if (gl == 0) red[warp * kMaxRowsPerGroup + rl] = dacc;
        __syncthreads();
        if (threadIdx.x < RB && r0 + threadIdx.x < rows) {
            const long long row = r0 + threadIdx.x;
            float tot = ep.d_in[row];
            for (int sl = 1; sl < ep.n_slots_in; ++sl) tot += ep.d_in[(size_t)sl * ep.slot_stride + row];
            for (int w2 = 0; w2 < kWarps; ++w2) tot += red[w2 * kMaxRowsPerGroup + threadIdx.x];
            if (EPI == CONVT_EPI_CONCRETIZE) {
                const int b2 = (int)(row / (2LL * ep.n_k)), up2 = (int)((row / ep.n_k) & 1), i2 = (int)(row % ep.n_k);
                CERT_ST((up2 ? ep.ub_out : ep.lb_out)[(size_t)b2 * ep.n_total + ep.out_off + i2], tot);
            } else {
                CERT_ST(ep.d_out[row], tot);
            }
        }
        if (EPI == CONVT_EPI_RELU) {
            // keep the padded tail of the rows at zero
            for (int q = 0; q < RB; ++q) {
                if (r0 + q >= rows) break;
                const size_t o = (size_t)(r0 + q) * ld_in;
                for (int t = n_in + threadIdx.x; t < ld_in; t += kThreads) {
                    CERT_ST(ep.P[o + t], 0.0f);
                    if (ep.P_lo) CERT_ST(ep.P_lo[o + t], 0.0f);
                }
            }
        }
    }
}

template <int CT, int PXT>
void launch_ct(const LayerDev &L, const ConvtPlan &pl, const float *Q, long long rows, int sms,
               const ConvtEpilogue &ep, cudaStream_t st) {
    long long groups = ceil_div_ll(rows, pl.rows_per_group);
    int grid = (int)std::min<long long>(groups, 2LL * sms);
    if (ep.mode == CONVT_EPI_CONCRETIZE)
        convt_kernel<CT, PXT, CONVT_EPI_CONCRETIZE><<<grid, kThreads, pl.smem_bytes, st>>>(
            Q, L.ld_out, L.ld_in, L.Wct, geom_of(L), pl, rows, ep);
    else
        convt_kernel<CT, PXT, CONVT_EPI_RELU><<<grid, kThreads, pl.smem_bytes, st>>>(
            Q, L.ld_out, L.ld_in, L.Wct, geom_of(L), pl, rows, ep);
}

template <int CT, int PXT>
void prepare_ct() {
    cudaFuncSetAttribute(convt_kernel<CT, PXT, CONVT_EPI_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kSmemBudget);
    cudaFuncSetAttribute(convt_kernel<CT, PXT, CONVT_EPI_CONCRETIZE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kSmemBudget);
}

template <int CT, int PXT, int T>
void launch_s2(const LayerDev &L, const ConvtPlan &pl, const float *Q, long long rows, int sms,
               const ConvtEpilogue &ep, cudaStream_t st) {
    long long groups = ceil_div_ll(rows, pl.rows_per_group);
    int grid = (int)std::min<long long>(groups, 2LL * sms);
    if (ep.mode == CONVT_EPI_CONCRETIZE)
        convt_s2_kernel<CT, PXT, T, CONVT_EPI_CONCRETIZE><<<grid, kThreads, pl.smem_bytes, st>>>(
            Q, L.ld_out, L.ld_in, L.Wct, geom_of(L), pl, rows, ep);
    else
        convt_s2_kernel<CT, PXT, T, CONVT_EPI_RELU><<<grid, kThreads, pl.smem_bytes, st>>>(
            Q, L.ld_out, L.ld_in, L.Wct, geom_of(L), pl, rows, ep);
}

template <int CT, int PXT>
void launch_s2_taps(const LayerDev &L, const ConvtPlan &pl, const float *Q, long long rows, int sms,
                    const ConvtEpilogue &ep, cudaStream_t st) {
    if (pl.ty == 1) launch_s2<CT, PXT, 1>(L, pl, Q, rows, sms, ep, st);
    else if (pl.ty == 2) launch_s2<CT, PXT, 2>(L, pl, Q, rows, sms, ep, st);
    else launch_s2<CT, PXT, 3>(L, pl, Q, rows, sms, ep, st);
}

template <int CT, int PXT, int T>
void prepare_s2() {
    cudaFuncSetAttribute(convt_s2_kernel<CT, PXT, T, CONVT_EPI_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kSmemBudget);
    cudaFuncSetAttribute(convt_s2_kernel<CT, PXT, T, CONVT_EPI_CONCRETIZE>,
                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
}

}  // namespace

// Whether the back-step through this conv layer fits the kernel's shared-memory plan.
bool convt_supported(const LayerDev &L) {
    if (L.stride > kMaxStride) return false;
    return make_plan(L).rows_per_group >= 1;
}

void convt_prepare() {
    prepare_s2<3, 5, 1>(); prepare_s2<3, 5, 2>(); prepare_s2<3, 5, 3>();
    prepare_s2<4, 4, 1>(); prepare_s2<4, 4, 2>(); prepare_s2<4, 4, 3>();
    prepare_ct<3, 8>();
    prepare_ct<4, 4>();
    prepare_ct<8, 4>();
    prepare_ct<16, 2>();
}

void launch_convt_ffma(const LayerDev &L, const float *Q, long long rows, int sms, const ConvtEpilogue &ep,
                       cudaStream_t st) {
    const ConvtPlan pl = make_plan(L);
    if (pl.s2) {
        if (L.c_in == 3) launch_s2_taps<3, 5>(L, pl, Q, rows, sms, ep, st);
        else launch_s2_taps<4, 4>(L, pl, Q, rows, sms, ep, st);
        return;
    }
    if (L.c_in == 3) launch_ct<3, 8>(L, pl, Q, rows, sms, ep, st);
    else if (L.c_in <= 4) launch_ct<4, 4>(L, pl, Q, rows, sms, ep, st);
    else if (L.c_in <= 8) launch_ct<8, 4>(L, pl, Q, rows, sms, ep, st);
    else launch_ct<16, 2>(L, pl, Q, rows, sms, ep, st);
}

}  // namespace cert
