// Conv back-steps on receptive-field patches.
//
// The expression of a conv neuron (co, oy, ox) of layer k over the outputs of a conv layer below is
// zero outside a window: the kernel's footprint, grown by (ph - 1) * stride + kernel at every further
// conv layer it is pushed through (the paper keeps such rows as convolution / patches blocks instead of
// dense ones, Section 5 and Appendix B).  While every layer between k and the end of the traversal is a
// conv layer and the window is smaller than the map, a row is held as the patch [C][ph][pw] plus the
// window's origin, which is a function of (oy, ox) alone:
//
//   level j (expression over the outputs of layer j):  origin_j = (oy, ox) * a_j - b_j
//   start (j = k-1):            ph = kh_k,                a = stride_k,      b = pad_k
//   through conv layer j:       ph' = (ph-1)*s_j + kh_j,  a' = a * s_j,      b' = b * s_j + pad_j
//
// In patch coordinates the back-step is a transposed convolution without padding,
//   out[ci][s*py + ky][s*px + kx] += in[co][py][px] * W[co][ci][ky][kx],
// and window positions that fall outside the image belong to no neuron: they carry no coefficient.
// The ReLU back-step below (replace_lower/upper) or the concretisation (map(simplify_*)) is applied
// to each element at its position in the image, exactly as in the dense kernels.
// One warp per row; row constants are warp-shuffle sums (fixed order).
#include "common.cuh"

namespace cert {

namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// replace_lower / replace_upper through a ReLU neuron with L = lamL*z, U = lamU*z + nuU.
__device__ __forceinline__ float relu_backstep(float c, int upper, float lamL, float lamU, float nuU,
                                               float &dacc) {
    const bool nonneg = (c >= 0.0f);
    const bool use_lower = upper ? !nonneg : nonneg;
    if (use_lower) return c * lamL;
    dacc = fmaf(c, nuU, dacc);
    return c * lamU;
}

// Start at conv layer k: patch over the layer's inputs = its kernel [c_in][kh][kw] at origin
// (oy*stride - pad, ox*stride - pad), pushed through the ReLU below; constant = bias + the nu terms +
// Q.b of the layer below.  Out-of-image window positions get 0.  With patch_lo the patch is written as a
// TF32 pair (hi in patch, lo in patch_lo) for a tensor-core step.
__device__ __forceinline__ float tf32_rn(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
patch_start_kernel(const float *__restrict__ Wk, ConvGeom gk, const float *__restrict__ bias_k,
                   float *__restrict__ patch, float *__restrict__ patch_lo, int pitch, float *__restrict__ d,
                   int n_k, int ld, int has_relu, const float *__restrict__ lamL, const float *__restrict__ lamU,
                   const float *__restrict__ nuU, const float *__restrict__ bias_below) {
    // One block per (box, output position): the window of the relaxation below is the same for the
    // 2 * c_out rows of that position, so it is looked up once and kept in shared memory.
    extern __shared__ __align__(16) float win[];
    float *sL = win, *sU = win + pitch, *sN = win + 2 * pitch, *sB = win + 3 * pitch;
    const int hw_o = gk.h_out * gk.w_out;
    const int box = blockIdx.x / hw_o, pos = blockIdx.x - box * hw_o;
    const int y0 = (pos / gk.w_out) * gk.stride - gk.pad, x0 = (pos % gk.w_out) * gk.stride - gk.pad;
    const int khw = gk.kh * gk.kw, taps = gk.c_in * khw;
    const size_t vec = (size_t)box * ld;
    for (int q = threadIdx.x; q < pitch; q += blockDim.x) {
        float l = 0.0f, u = 0.0f, n = 0.0f, bz = 0.0f;
        if (q < taps) {
            const int ci = q / khw, ky = (q / gk.kw) % gk.kh, kx = q % gk.kw;
            const int iy = y0 + ky, ix = x0 + kx;
            if (iy >= 0 && iy < gk.h_in && ix >= 0 && ix < gk.w_in) {
                const int t = (ci * gk.h_in + iy) * gk.w_in + ix;
                l = has_relu ? lamL[vec + t] : 1.0f;
                u = has_relu ? lamU[vec + t] : 1.0f;
                n = has_relu ? nuU[vec + t] : 0.0f;
                bz = bias_below[t];
            }
        }
        sL[q] = l; sU[q] = u; sN[q] = n; sB[q] = bz;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rr = warp; rr < 2 * gk.c_out; rr += kWarpsPerBlock) {
        const int upper = rr / gk.c_out, co = rr - upper * gk.c_out;
        const int i = co * hw_o + pos;
        // tensor-core steps follow (patch_lo): rows ordered (box, position, side, channel); else (box, side, neuron)
        const long long r = patch_lo ? (long long)blockIdx.x * 2 * gk.c_out + rr
                                     : ((long long)box * 2 + upper) * n_k + i;
        const float *wrow = Wk + (size_t)co * taps;
        float dacc = 0.0f;
        for (int q0 = lane * 4; q0 < pitch; q0 += 128) {
            const float4 l4 = *reinterpret_cast<const float4 *>(sL + q0);
            const float4 u4 = *reinterpret_cast<const float4 *>(sU + q0);
            const float4 n4 = *reinterpret_cast<const float4 *>(sN + q0);
            const float4 b4 = *reinterpret_cast<const float4 *>(sB + q0);
            const float la[4] = {l4.x, l4.y, l4.z, l4.w}, ua[4] = {u4.x, u4.y, u4.z, u4.w};
            const float na[4] = {n4.x, n4.y, n4.z, n4.w}, ba[4] = {b4.x, b4.y, b4.z, b4.w};
            float qv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float c = (q0 + e < taps) ? wrow[q0 + e] : 0.0f;
                qv[e] = relu_backstep(c, upper, la[e], ua[e], na[e], dacc);   // zero outside the map
                dacc = fmaf(qv[e], ba[e], dacc);
            }
            float *dst = patch + (size_t)r * pitch + q0;
            if (patch_lo) {
                float h[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    h[e] = tf32_rn(qv[e]);
                    lo[e] = tf32_rn(qv[e] - h[e]);
                }
                CERT_ST(*reinterpret_cast<float4 *>(dst), make_float4(h[0], h[1], h[2], h[3]));
                CERT_ST(*reinterpret_cast<float4 *>(patch_lo + (size_t)r * pitch + q0), make_float4(lo[0], lo[1], lo[2], lo[3]));
            } else {
                CERT_ST(*reinterpret_cast<float4 *>(dst), make_float4(qv[0], qv[1], qv[2], qv[3]));
            }
        }
        dacc = warp_sum(dacc);
        if (lane == 0) CERT_ST(d[r], bias_k[i] + dacc);
    }
}

// Per (box, output position of the conv neuron): the window of up to three per-neuron arrays of the
// layer the window lies in, laid out like the patch ([c][qh][qw], zero padded to ld_dst); positions
// outside the map get 0, so that they drop out of whatever the values multiply.  A null source
// stands for the constant fill[i] inside the map (no ReLU below: slopes 1, intercept 0).
struct PatchGather {
    int c, qh, qw;         // window
    int h, w;              // map of the layer the window lies in
    int a, b;              // window origin = (oy, ox) * a - b
    int w_k, n_pos;        // layer k's output map: width, positions
    int ld_src, ld_dst;
    int n_arr;
    const float *src[3];
    float fill[3];
    float *dst[3];
};

__global__ void patch_gather_kernel(const PatchGather g) {
    const int v = blockIdx.x;                    // box * n_pos + position
    const int box = v / g.n_pos, pos = v - box * g.n_pos;
    const int gy0 = (pos / g.w_k) * g.a - g.b, gx0 = (pos % g.w_k) * g.a - g.b;
    const int qhw = g.qh * g.qw, elems = g.c * qhw;
    for (int e = threadIdx.x; e < g.ld_dst; e += blockDim.x) {
        int t = -1;
        if (e < elems) {
            const int ci = e / qhw, rem = e - ci * qhw;
            const int gy = gy0 + rem / g.qw, gx = gx0 + rem % g.qw;
            if (gy >= 0 && gy < g.h && gx >= 0 && gx < g.w) t = (ci * g.h + gy) * g.w + gx;
        }
        for (int i = 0; i < g.n_arr; ++i) {
            float val = 0.0f;
            if (t >= 0) val = g.src[i] ? g.src[i][(size_t)box * g.ld_src + t] : g.fill[i];
            CERT_ST(g.dst[i][(size_t)v * g.ld_dst + e], val);
        }
    }
}

// Geometry of one patch back-step through conv layer j for the rows of conv layer k.
struct PatchStep {
    int ph, pw;              // input patch (over the outputs of layer j): [c_out][ph][pw]
    int qh, qw;              // output patch (over the inputs of layer j): [c_in][qh][qw], qh = (ph-1)*s + kh
    int pitch_in, pitch_out; // floats per row of the patch buffers
    int a, b;                // origin of the output patch = (oy, ox) * a - b
    int hw_k, w_k;           // layer k's output map h*w and w (decode neuron -> (oy, ox))
};

// Shared memory: weights [c_out][c_in][kh][kw]; index tables (built once per block, so that the row loop has
// no divisions): pix[p] = (y << 16) | x of output pixel p; for every output row y the taps (ky << 16) | py with
// y = s*py + ky, 0 <= py < ph, ky < kh (count in ycnt[y]), the same for columns; then one input patch per warp.
__host__ __device__ inline int patch_taps_max(int k, int s) { return (k + s - 1) / s; }
__host__ __device__ inline int patch_table_ints(const ConvGeom &g, int qh, int qw) {
    return qh * qw + qh * (patch_taps_max(g.kh, g.stride) + 1) + qw * (patch_taps_max(g.kw, g.stride) + 1);
}

template <int EPI>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
patch_step_kernel(const float *__restrict__ in, const float *__restrict__ W, ConvGeom g, PatchStep ps,
                  long long rows, int ld_in, ConvtEpilogue ep) {
    extern __shared__ __align__(16) float smem[];
    const int n_w = g.c_out * g.c_in * g.kh * g.kw;
    const int n_inp = g.c_out * ps.ph * ps.pw;
    const int s = g.stride;
    const int tym = patch_taps_max(g.kh, s), txm = patch_taps_max(g.kw, s);
    float *Ws = smem;
    int *pix = reinterpret_cast<int *>(smem + n_w);
    int *ycnt = pix + ps.qh * ps.qw, *ytab = ycnt + ps.qh;
    int *xcnt = ytab + ps.qh * tym, *xtab = xcnt + ps.qw;
    float *my_patch = reinterpret_cast<float *>(xtab + ps.qw * txm) + (threadIdx.x >> 5) * n_inp;
    for (int i = threadIdx.x; i < n_w; i += blockDim.x) Ws[i] = W[i];
    for (int p = threadIdx.x; p < ps.qh * ps.qw; p += blockDim.x) pix[p] = ((p / ps.qw) << 16) | (p % ps.qw);
    for (int y = threadIdx.x; y < ps.qh; y += blockDim.x) {
        int n = 0;
        for (int ky = y % s; ky < g.kh && ky <= y; ky += s)
            if ((y - ky) / s < ps.ph) ytab[y * tym + n++] = (ky << 16) | ((y - ky) / s);
        ycnt[y] = n;
    }
    for (int x = threadIdx.x; x < ps.qw; x += blockDim.x) {
        int n = 0;
        for (int kx = x % s; kx < g.kw && kx <= x; kx += s)
            if ((x - kx) / s < ps.pw) xtab[x * txm + n++] = (kx << 16) | ((x - kx) / s);
        xcnt[x] = n;
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * kWarpsPerBlock;
    const int khw = g.kh * g.kw, w_co = g.c_in * khw;
    const int phw = ps.ph * ps.pw, qhw = ps.qh * ps.qw;
    const int n_outp = g.c_in * qhw;
    const int hw_in = g.h_in * g.w_in;

    for (long long r = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); r < rows; r += warps_total) {
        __syncwarp();
        const float *irow = in + (size_t)r * ps.pitch_in;
        for (int e = lane; e < n_inp; e += 32) my_patch[e] = irow[e];
        __syncwarp();

        const int box = (int)(r / (2LL * ep.n_k));
        const int upper = (int)((r / ep.n_k) & 1);
        const int i = (int)(r % ep.n_k);
        const int oy = (i / ps.w_k) % (ps.hw_k / ps.w_k), ox = i % ps.w_k;
        const int gy0 = oy * ps.a - ps.b, gx0 = ox * ps.a - ps.b;      // origin of the output patch in the image
        const size_t vec = (size_t)box * ld_in;
        float dacc = 0.0f;
        for (int e = lane; e < n_outp; e += 32) {
            const int ci = e / qhw;
            const int yx = pix[e - ci * qhw];
            const int y = yx >> 16, x = yx & 0xffff;
            const int gy = gy0 + y, gx = gx0 + x;
            const bool inside = gy >= 0 && gy < g.h_in && gx >= 0 && gx < g.w_in;
            float acc = 0.0f;
            if (inside) {
                const int ny = ycnt[y], nx = xcnt[x];
                for (int a = 0; a < ny; ++a) {
                    const int yt = ytab[y * tym + a];
                    const int ky = yt >> 16, py = yt & 0xffff;
                    for (int b2 = 0; b2 < nx; ++b2) {
                        const int xt = xtab[x * txm + b2];
                        const int kx = xt >> 16, px = xt & 0xffff;
                        const float *ip = my_patch + py * ps.pw + px;
                        const float *wp = Ws + (ci * g.kh + ky) * g.kw + kx;
#pragma unroll 4
                        for (int co = 0; co < g.c_out; ++co) acc = fmaf(ip[co * phw], wp[co * w_co], acc);
                    }
                }
                const int t = ci * hw_in + gy * g.w_in + gx;
                if (EPI == CONVT_EPI_CONCRETIZE) {
                    const bool nonneg = (acc >= 0.0f);
                    dacc = fmaf(acc, (nonneg != (upper != 0)) ? ep.l0[vec + t] : ep.u0[vec + t], dacc);
                } else {
                    if (ep.has_relu) acc = relu_backstep(acc, upper, ep.lamL[vec + t], ep.lamU[vec + t], ep.nuU[vec + t], dacc);
                    dacc = fmaf(acc, ep.bias_below[t], dacc);
                }
            }
            if (EPI == CONVT_EPI_RELU) CERT_ST(ep.P[(size_t)r * ps.pitch_out + e], acc);
        }
        if (EPI == CONVT_EPI_RELU) {
            for (int e = n_outp + lane; e < ps.pitch_out; e += 32) CERT_ST(ep.P[(size_t)r * ps.pitch_out + e], 0.0f);
        }
        dacc = warp_sum(dacc);
        if (lane == 0) {
            float tot = ep.d_in[r];
            for (int sl = 1; sl < ep.n_slots_in; ++sl) tot += ep.d_in[(size_t)sl * ep.slot_stride + r];
            tot += dacc;
            if (EPI == CONVT_EPI_CONCRETIZE)
                CERT_ST((upper ? ep.ub_out : ep.lb_out)[(size_t)box * ep.n_total + ep.out_off + i], tot);
            else
                CERT_ST(ep.d_out[r], tot);
        }
    }
}

}  // namespace

constexpr size_t kPatchSmemMax = 96 * 1024;

static size_t patch_step_smem(const LayerDev &Lj, const PatchLevel &in) {
    const int qh = (in.ph - 1) * Lj.stride + Lj.kh, qw = (in.pw - 1) * Lj.stride + Lj.kw;
    return sizeof(float) * ((size_t)Lj.c_out * Lj.c_in * Lj.kh * Lj.kw + (size_t)patch_table_ints(geom_of(Lj), qh, qw) +
                            (size_t)kWarpsPerBlock * in.elems);
}

bool conv_patch_plan(const LayerDev *layers, int k, int j_end, PatchLevel *levels, int max_levels) {
    const LayerDev &Lk = layers[k];
    if (Lk.kind != CERT_LAYER_CONV2D || k - j_end + 1 > max_levels) return false;
    PatchLevel lv;
    lv.c = Lk.c_in; lv.ph = Lk.kh; lv.pw = Lk.kw; lv.a = Lk.stride; lv.b = Lk.pad;
    lv.elems = lv.c * lv.ph * lv.pw;
    lv.pitch = round_up(lv.elems, 4);
    if (2 * lv.elems > Lk.n_in) return false;            // the window is not much smaller than the map
    if (16 * (size_t)round_up(lv.elems, kPad) > 48 * 1024) return false;   // the start kernel's shared-memory window
    levels[0] = lv;
    for (int j = k - 1, m = 1; j >= j_end; --j, ++m) {
        const LayerDev &Lj = layers[j];
        if (Lj.kind != CERT_LAYER_CONV2D) return false;
        if (patch_step_smem(Lj, levels[m - 1]) > kPatchSmemMax) return false;
        PatchLevel nx;
        nx.c = Lj.c_in;
        nx.ph = (levels[m - 1].ph - 1) * Lj.stride + Lj.kh;
        nx.pw = (levels[m - 1].pw - 1) * Lj.stride + Lj.kw;
        nx.a = levels[m - 1].a * Lj.stride;
        nx.b = levels[m - 1].b * Lj.stride + Lj.pad;
        nx.elems = nx.c * nx.ph * nx.pw;
        nx.pitch = round_up(nx.elems, 4);
        if (2 * nx.elems > Lj.n_in) return false;
        levels[m] = nx;
    }
    return true;
}

void conv_patch_prepare() {
    cudaFuncSetAttribute(patch_step_kernel<CONVT_EPI_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kPatchSmemMax);
    cudaFuncSetAttribute(patch_step_kernel<CONVT_EPI_CONCRETIZE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kPatchSmemMax);
}

void launch_patch_start(const LayerDev &Lk, const LayerDev &Lb, int pitch, int batch, float *patch,
                        float *patch_lo, float *d, cudaStream_t st) {
    const unsigned grid = (unsigned)(batch * Lk.h_out * Lk.w_out);
    patch_start_kernel<<<grid, kWarpsPerBlock * 32, 4 * (size_t)pitch * sizeof(float), st>>>(
        Lk.W, geom_of(Lk), Lk.bias_n, patch, patch_lo, pitch, d, Lk.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL, Lb.lamU,
        Lb.nuU, Lb.bias_n);
}

// ---- y-major copies for the banded tensor-core form of the dense conv back-steps ----
// A map [c][h][w] (flattened channel-major, as everywhere else) reordered to [h][c][w], so that a band of map
// rows is one contiguous piece of the row.

// Coefficient matrix (TF32 pair) of `rows` rows: dst[r][(y*c + ch)*w + x] = src[r][(ch*h + y)*w + x].
__global__ void to_ymajor_pair_kernel(const float *__restrict__ src_hi, const float *__restrict__ src_lo,
                                      float *__restrict__ dst_hi, float *__restrict__ dst_lo, long long rows, int c,
                                      int h, int w, int ld) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int n = c * h * w;
    if (idx >= rows * (long long)n) return;
    const long long r = idx / n;
    const int e = (int)(idx - r * n);
    const int y = e / (c * w), rem = e - y * (c * w);
    const int ch = rem / w, x = rem - ch * w;
    const size_t s = (size_t)r * ld + (size_t)(ch * h + y) * w + x;
    CERT_ST(dst_hi[(size_t)r * ld + e], src_hi[s]);
    CERT_ST(dst_lo[(size_t)r * ld + e], src_lo[s]);
}

// Up to three per-neuron arrays [batch][ld]; a null source stands for fill[i].
struct YMajorVectors {
    int c, h, w, ld, n_arr;
    const float *src[3];
    float fill[3];
    float *dst[3];
};

__global__ void to_ymajor_vectors_kernel(const YMajorVectors g, int batch) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int n = g.c * g.h * g.w;
    if (idx >= (long long)batch * n) return;
    const int b = (int)(idx / n), e = (int)(idx - (long long)b * n);
    const int y = e / (g.c * g.w), rem = e - y * (g.c * g.w);
    const int ch = rem / g.w, x = rem - ch * g.w;
    const size_t s = (size_t)b * g.ld + (size_t)(ch * g.h + y) * g.w + x;
    for (int i = 0; i < g.n_arr; ++i) CERT_ST(g.dst[i][(size_t)b * g.ld + e], g.src[i] ? g.src[i][s] : g.fill[i]);
}

void launch_to_ymajor_pair(const float *src_hi, const float *src_lo, float *dst_hi, float *dst_lo, long long rows,
                           int c, int h, int w, int ld, cudaStream_t st) {
    const long long total = rows * (long long)c * h * w;
    to_ymajor_pair_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(src_hi, src_lo, dst_hi, dst_lo, rows, c, h,
                                                                           w, ld);
}

void launch_to_ymajor_vectors(int c, int h, int w, int ld, int batch, int n_arr, const float *const *src,
                              const float *fill, float *const *dst, cudaStream_t st) {
    YMajorVectors g;
    g.c = c; g.h = h; g.w = w; g.ld = ld; g.n_arr = n_arr;
    for (int i = 0; i < 3; ++i) {
        g.src[i] = i < n_arr ? src[i] : nullptr;
        g.fill[i] = i < n_arr ? fill[i] : 0.0f;
        g.dst[i] = i < n_arr ? dst[i] : nullptr;
    }
    const long long total = (long long)batch * c * h * w;
    to_ymajor_vectors_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(g, batch);
}

void launch_patch_gather(const LayerDev &Lk, const LayerDev &Lj, const PatchLevel &out, int ld_dst, int batch,
                         int n_arr, const float *const *src, const float *fill, float *const *dst,
                         cudaStream_t st) {
    PatchGather g;
    g.c = out.c; g.qh = out.ph; g.qw = out.pw;
    g.h = Lj.h_in; g.w = Lj.w_in;
    g.a = out.a; g.b = out.b;
    g.w_k = Lk.w_out; g.n_pos = Lk.h_out * Lk.w_out;
    g.ld_src = Lj.ld_in; g.ld_dst = ld_dst;
    g.n_arr = n_arr;
    for (int i = 0; i < 3; ++i) {
        g.src[i] = i < n_arr ? src[i] : nullptr;
        g.fill[i] = i < n_arr ? fill[i] : 0.0f;
        g.dst[i] = i < n_arr ? dst[i] : nullptr;
    }
    patch_gather_kernel<<<(unsigned)(batch * g.n_pos), 128, 0, st>>>(g);
}

void launch_patch_step(const LayerDev &Lk, const LayerDev &Lj, const PatchLevel &in, const PatchLevel &out,
                       const float *in_patch, long long rows, int sms, const ConvtEpilogue &ep, cudaStream_t st) {
    PatchStep ps;
    ps.ph = in.ph; ps.pw = in.pw; ps.qh = out.ph; ps.qw = out.pw;
    ps.pitch_in = in.pitch; ps.pitch_out = out.pitch;
    ps.a = out.a; ps.b = out.b;
    ps.hw_k = Lk.h_out * Lk.w_out; ps.w_k = Lk.w_out;
    const size_t smem = patch_step_smem(Lj, in);
    const long long blocks_needed = ceil_div_ll(rows, kWarpsPerBlock);
    const int grid = (int)std::min<long long>(blocks_needed, 8LL * sms);
    if (ep.mode == CONVT_EPI_CONCRETIZE)
        patch_step_kernel<CONVT_EPI_CONCRETIZE><<<grid, kWarpsPerBlock * 32, smem, st>>>(in_patch, Lj.W, geom_of(Lj), ps,
                                                                                      rows, Lj.ld_in, ep);
    else
        patch_step_kernel<CONVT_EPI_RELU><<<grid, kWarpsPerBlock * 32, smem, st>>>(in_patch, Lj.W, geom_of(Lj), ps, rows,
                                                                                Lj.ld_in, ep);
}

}  // namespace cert
