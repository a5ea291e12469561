// Conv back-step: a row's coefficient map over the outputs of a conv layer is
// pushed through the layer by the exact transpose of the convolution
// (Appendix B: a dense block times a convolution block is conv_transpose2d):
//
//   P[r][ci][iy][ix] = sum over (co, ky, kx) with (iy + pad - ky) = stride * oy and
//                      (ix + pad - kx) = stride * ox of  Q[r][co][oy][ox] * W[co][ci][ky][kx]
//
// Implicit GEMM on the fp32 FMA units (the channel count below a conv layer is
// 3..16: too narrow an N for the tensor cores).  Input pixels fall into
// stride x stride classes by ((iy + pad) mod stride, (ix + pad) mod stride);
// every pixel of a class uses the same kernel taps, so a warp that works on one
// class reads its weights as warp-uniform 16-byte shared-memory loads.  A block
// stages the maps of a group of rows in shared memory inside a zero halo (no
// bounds tests in the inner loop); a thread accumulates PXT pixels x CT
// channels in registers, so a coefficient read from shared memory feeds CT
// FMAs and a weight PXT FMAs.
#include "common.cuh"

namespace cert {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int PXT = 4;                       // pixels per thread
constexpr int kMaxStride = 4;
constexpr size_t kSmemBudget = 200 * 1024;

// Shared-memory plan of one conv layer's back-step, derived on the host.
struct ConvtPlan {
    int halo_y, halo_x;      // zero rows / columns before the map
    int HP, WP;              // padded map height / width
    int map_stride;          // floats between consecutive rows' staged maps
    int cpad;                // c_in rounded up to 4 (weights are staged as [co][ky][kx][cpad])
    int rows_per_group;      // rows staged per pass
    size_t smem_bytes;
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
    // Pixels per class row; consecutive lanes walk them and then move to the next staged row, so a map
    // stride congruent to that count modulo 32 keeps a warp's loads on distinct banks.
    int wc = (L.w_in + L.stride - 1) / L.stride;
    int ms = L.c_out * p.HP * p.WP;
    while (ms % 32 != wc % 32) ++ms;
    p.map_stride = ms;
    p.cpad = round_up(L.c_in, 4);
    size_t w_bytes = sizeof(float) * (size_t)L.c_out * L.kh * L.kw * p.cpad;
    size_t per_row = sizeof(float) * (size_t)ms;
    long long fit = w_bytes < kSmemBudget ? (long long)((kSmemBudget - w_bytes) / per_row) : 0;
    p.rows_per_group = (int)std::min<long long>(fit, 16);
    p.smem_bytes = w_bytes + per_row * (size_t)std::max(p.rows_per_group, 1);
    return p;
}

// Q [rows][ld_out] maps (c_out, h_out, w_out); P [rows][ld_in] maps (c_in, h_in, w_in).
// Wct: weights laid out [c_out][kh][kw][c_in].
template <int CT>
__global__ void __launch_bounds__(kThreads, 1)
convt_kernel(const float *__restrict__ Q, int ld_out, float *__restrict__ P, int ld_in,
             const float *__restrict__ Wct, ConvGeom g, ConvtPlan pl, long long rows) {
    extern __shared__ __align__(16) float smem[];
    const int n_out = g.c_out * g.h_out * g.w_out;
    const int n_in = g.c_in * g.h_in * g.w_in;
    const int hw_in = g.h_in * g.w_in, hw_out = g.h_out * g.w_out;
    const int n_w = g.c_out * g.kh * g.kw * pl.cpad;
    const int RB = pl.rows_per_group;
    const int plane = pl.HP * pl.WP;
    float *Ws = smem;                  // [c_out][kh][kw][cpad]
    float *Qs = smem + n_w;            // [RB][map_stride], each map [c_out][HP][WP] inside its halo
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < n_w; i += kThreads) {
        int ci = i % pl.cpad, tap = i / pl.cpad;
        Ws[i] = ci < g.c_in ? Wct[(size_t)tap * g.c_in + ci] : 0.0f;
    }
    for (int i = threadIdx.x; i < RB * pl.map_stride; i += kThreads) Qs[i] = 0.0f;   // halos stay zero

    const int s = g.stride;
    const int n_classes = s * s;

    for (long long r0 = (long long)blockIdx.x * RB; r0 < rows; r0 += (long long)gridDim.x * RB) {
        __syncthreads();
        // stage the maps of rows r0 .. r0+RB-1 (rows past the end read as zero); the element index
        // advances by the block size, its (co, oy, ox) decomposition with it
        {
            const int d_ox = kThreads % g.w_out, d_oy = (kThreads / g.w_out) % g.h_out, d_co = kThreads / hw_out;
            for (int rl = 0; rl < RB; ++rl) {
                const bool live = r0 + rl < rows;
                const float *qrow = Q + (size_t)(r0 + rl) * ld_out;
                float *qs = Qs + rl * pl.map_stride + pl.halo_y * pl.WP + pl.halo_x;
                int e = threadIdx.x;
                int co = e / hw_out, oy = (e % hw_out) / g.w_out, ox = e % g.w_out;
                for (; e < n_out; e += kThreads) {
                    qs[co * plane + oy * pl.WP + ox] = live ? qrow[e] : 0.0f;
                    ox += d_ox;
                    if (ox >= g.w_out) { ox -= g.w_out; ++oy; }
                    oy += d_oy;
                    if (oy >= g.h_out) { oy -= g.h_out; ++co; }
                    co += d_co;
                }
            }
        }
        __syncthreads();

        // Work units: (class, chunk of 32*PXT items); an item is (row of the group, pixel of the class).
        int unit_base = 0;
        for (int cls = 0; cls < n_classes; ++cls) {
            const int cy = cls / s, cx = cls % s;
            // pixels of the class: iy = cy - pad + s*uy, 0 <= iy < h_in; then oy = uy - my for ky = cy + s*my
            const int uy0 = (g.pad - cy + s - 1 >= 0) ? (g.pad - cy + s - 1) / s : 0;
            const int ux0 = (g.pad - cx + s - 1 >= 0) ? (g.pad - cx + s - 1) / s : 0;
            const int uy1 = (g.h_in - 1 + g.pad - cy >= 0) ? (g.h_in - 1 + g.pad - cy) / s : -1;
            const int ux1 = (g.w_in - 1 + g.pad - cx >= 0) ? (g.w_in - 1 + g.pad - cx) / s : -1;
            const int Hc = uy1 - uy0 + 1, Wc = ux1 - ux0 + 1;
            const int n_my = cy < g.kh ? (g.kh - cy + s - 1) / s : 0;
            const int n_mx = cx < g.kw ? (g.kw - cx + s - 1) / s : 0;
            if (Hc <= 0 || Wc <= 0) continue;
            const int items = Hc * RB * Wc;
            const int units = (items + 32 * PXT - 1) / (32 * PXT);
            // warps take units round-robin across classes
            int first = ((warp - unit_base) % kWarps + kWarps) % kWarps;
            for (int u = first; u < units; u += kWarps) {
                int q_off[PXT], p_off[PXT];
                long long p_row[PXT];
#pragma unroll
                for (int i = 0; i < PXT; ++i) {
                    int it = u * (32 * PXT) + i * 32 + lane;
                    bool ok = it < items;
                    int itc = ok ? it : 0;
                    int ux = itc % Wc, t2 = itc / Wc, rl = t2 % RB, uy = t2 / RB;
                    q_off[i] = rl * pl.map_stride + (uy0 + uy + pl.halo_y) * pl.WP + (ux0 + ux + pl.halo_x);
                    int iy = cy - g.pad + s * (uy0 + uy), ix = cx - g.pad + s * (ux0 + ux);
                    p_off[i] = iy * g.w_in + ix;
                    p_row[i] = (ok && r0 + rl < rows) ? r0 + rl : -1;
                }
                for (int c0 = 0; c0 < g.c_in; c0 += CT) {
                    float acc[PXT][CT];
#pragma unroll
                    for (int i = 0; i < PXT; ++i)
#pragma unroll
                        for (int c = 0; c < CT; ++c) acc[i][c] = 0.0f;
                    for (int co = 0; co < g.c_out; ++co) {
                        for (int my = 0; my < n_my; ++my) {
                            const int ky = cy + s * my;
                            for (int mx = 0; mx < n_mx; ++mx) {
                                const int kx = cx + s * mx;
                                const float *wp = Ws + ((co * g.kh + ky) * g.kw + kx) * pl.cpad + c0;
                                float w[CT];
#pragma unroll
                                for (int c4 = 0; c4 < CT; c4 += 4) {
                                    // cpad is a multiple of 4; channels past cpad (CT > remaining) are skipped
                                    float4 w4 = (c0 + c4 < pl.cpad) ? *reinterpret_cast<const float4 *>(wp + c4)
                                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
                                    w[c4] = w4.x; w[c4 + 1] = w4.y; w[c4 + 2] = w4.z; w[c4 + 3] = w4.w;
                                }
                                const int shift = co * plane - my * pl.WP - mx;
#pragma unroll
                                for (int i = 0; i < PXT; ++i) {
                                    const float q = Qs[q_off[i] + shift];
#pragma unroll
                                    for (int c = 0; c < CT; ++c) acc[i][c] = fmaf(q, w[c], acc[i][c]);
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int i = 0; i < PXT; ++i) {
                        if (p_row[i] < 0) continue;
                        float *prow = P + (size_t)p_row[i] * ld_in + p_off[i];
#pragma unroll
                        for (int c = 0; c < CT; ++c)
                            if (c0 + c < g.c_in) prow[(size_t)(c0 + c) * hw_in] = acc[i][c];
                    }
                }
            }
            unit_base += units;
        }
        // keep the padded tail of the rows at zero
        for (int rl = 0; rl < RB; ++rl) {
            if (r0 + rl >= rows) break;
            float *prow = P + (size_t)(r0 + rl) * ld_in;
            for (int t = n_in + threadIdx.x; t < ld_in; t += kThreads) prow[t] = 0.0f;
        }
    }
}

template <int CT>
void launch_ct(const LayerDev &L, const ConvtPlan &pl, const float *Q, float *P, long long rows, int sms,
               cudaStream_t st) {
    long long groups = ceil_div_ll(rows, pl.rows_per_group);
    int grid = (int)std::min<long long>(groups, sms);
    convt_kernel<CT><<<grid, kThreads, pl.smem_bytes, st>>>(Q, L.ld_out, P, L.ld_in, L.Wct, geom_of(L), pl, rows);
}

}  // namespace

// Whether the back-step through this conv layer fits the kernel's shared-memory plan.
bool convt_supported(const LayerDev &L) {
    if (L.stride > kMaxStride) return false;
    return make_plan(L).rows_per_group >= 1;
}

void convt_prepare() {
    cudaFuncSetAttribute(convt_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    cudaFuncSetAttribute(convt_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    cudaFuncSetAttribute(convt_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
}

void launch_convt_ffma(const LayerDev &L, const float *Q, float *P, long long rows, int sms, cudaStream_t st) {
    const ConvtPlan pl = make_plan(L);
    if (L.c_in <= 4) launch_ct<4>(L, pl, Q, P, rows, sms, st);
    else if (L.c_in <= 8) launch_ct<8>(L, pl, Q, P, rows, sms, st);
    else launch_ct<16>(L, pl, Q, P, rows, sms, st);
}

}  // namespace cert
