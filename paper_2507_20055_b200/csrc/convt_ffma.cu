// Conv back-step: a row's coefficient map over the outputs of a conv layer is
// pushed through the layer by the exact transpose of the convolution
// (Appendix B: a dense block times a convolution block is conv_transpose2d).
// Gather form on the fp32 FMA units: each block stages a few rows' maps in
// shared memory, each thread owns one input pixel and all its channels.
#include "common.cuh"

namespace cert {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxCin = 16;   // channels accumulated per pass

// Q [rows][ld_out] maps (c_out, h_out, w_out); P [rows][ld_in] maps (c_in, h_in, w_in).
// Wct: weights re-laid as [c_out][kh][kw][c_in].
__global__ void __launch_bounds__(kThreads)
convt_kernel(const float *__restrict__ Q, int ld_out, float *__restrict__ P, int ld_in,
             const float *__restrict__ Wct, ConvGeom g, long long rows) {
    extern __shared__ float smem[];
    const int n_out = g.c_out * g.h_out * g.w_out;
    const int n_in = g.c_in * g.h_in * g.w_in;
    const int n_w = g.c_out * g.kh * g.kw * g.c_in;
    float *Ws = smem;                 // [c_out][kh][kw][c_in]
    float *Qs = smem + n_w;           // [n_out]
    for (int i = threadIdx.x; i < n_w; i += kThreads) Ws[i] = Wct[i];
    const int hw_in = g.h_in * g.w_in, hw_out = g.h_out * g.w_out;

    for (long long r = blockIdx.x; r < rows; r += gridDim.x) {
        __syncthreads();
        const float *qrow = Q + (size_t)r * ld_out;
        for (int i = threadIdx.x; i < n_out; i += kThreads) Qs[i] = qrow[i];
        __syncthreads();
        float *prow = P + (size_t)r * ld_in;
        for (int c0 = 0; c0 < g.c_in; c0 += kMaxCin) {
            const int nc = min(kMaxCin, g.c_in - c0);
            for (int pix = threadIdx.x; pix < hw_in; pix += kThreads) {
                const int iy = pix / g.w_in, ix = pix % g.w_in;
                float acc[kMaxCin];
#pragma unroll
                for (int c = 0; c < kMaxCin; ++c) acc[c] = 0.0f;
                for (int ky = 0; ky < g.kh; ++ky) {
                    int ty = iy + g.pad - ky;
                    if (ty < 0 || ty % g.stride != 0) continue;
                    int oy = ty / g.stride;
                    if (oy >= g.h_out) continue;
                    for (int kx = 0; kx < g.kw; ++kx) {
                        int tx = ix + g.pad - kx;
                        if (tx < 0 || tx % g.stride != 0) continue;
                        int ox = tx / g.stride;
                        if (ox >= g.w_out) continue;
                        const float *qs = Qs + oy * g.w_out + ox;
                        const float *ws = Ws + (ky * g.kw + kx) * g.c_in + c0;
                        for (int co = 0; co < g.c_out; ++co) {
                            float q = qs[co * hw_out];
                            const float *w = ws + (size_t)co * g.kh * g.kw * g.c_in;
#pragma unroll
                            for (int c = 0; c < kMaxCin; ++c)
                                if (c < nc) acc[c] = fmaf(q, w[c], acc[c]);
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < kMaxCin; ++c)
                    if (c < nc) prow[(c0 + c) * hw_in + pix] = acc[c];
            }
        }
        // keep the padded tail of the row at zero
        for (int t = n_in + threadIdx.x; t < ld_in; t += kThreads) prow[t] = 0.0f;
    }
}

}  // namespace

size_t convt_smem_bytes(const LayerDev &L) {
    return sizeof(float) * ((size_t)L.c_out * L.kh * L.kw * L.c_in + (size_t)L.n_out);
}

void convt_prepare() {
    cudaFuncSetAttribute(convt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

void launch_convt_ffma(const LayerDev &L, const float *Q, float *P, long long rows, cudaStream_t st) {
    size_t smem = convt_smem_bytes(L);
    long long grid = rows < 148 * 4 ? rows : 148 * 4;
    convt_kernel<<<(unsigned)grid, kThreads, smem, st>>>(Q, L.ld_out, P, L.ld_in, L.Wct, geom_of(L), rows);
}

}  // namespace cert
