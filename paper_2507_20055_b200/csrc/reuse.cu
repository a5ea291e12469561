// Bandwidth-bound steps of the ReuseCert certifier (Appendix C, ReuseCert listing; Section 6.1):
// every neuron's polyhedral bounds L, U are kept over the input layer and reused, so an affine layer
// needs one contraction instead of a traversal.
//
// Layout.  The shapes of a layer's outputs (after its ReLU) are one matrix S per layer:
//   row (box, s):  s < n0 the coefficient of input x_s, s == n0 the constant, then zero rows up to
//                  R = rows per box (a multiple of 32);
//   column t < n:  lower shape L_t,  column n + t: upper shape U_t,  zero columns up to the pitch.
// With that layout "replace every ReLU neuron below by its stored L / U" (replace_lower/upper) is
//   [L_k | U_k] = S_{k-1} * [[W+^T, W-^T], [W-^T, W+^T]]   (+ the bias on the constant row),
// one contraction per affine layer with rows = boxes x R, which the fp16-split tensor-core kernel runs; its
// epilogue also leaves, per 32 rows, every column's concretisation terms (map(simplify_*)).
// The kernels here start the chain, turn those sums into bounds and relaxations (Relu transformer:
// relu_n, compute_upper on l = L.map(simplify_lower), u = U.map(simplify_upper)), and scale the raw
// [L_k | U_k] into S_k.
#include <cuda_fp16.h>

#include "common.cuh"

namespace cert {

namespace {

// Bounds of layer k from the column sums the contraction left (R/32 partial sums per box and column,
// added in order), then the Relu transformer.  One thread per (box, padded neuron).
__global__ void reuse_relax_kernel(const float *__restrict__ colsum, int ld_s, int groups_per_box, int n, int ld,
                                   int batch, float *__restrict__ lb_out, float *__restrict__ ub_out, int n_total,
                                   int out_off, int do_relax, float *__restrict__ lamL, float *__restrict__ lamU,
                                   float *__restrict__ nuU, unsigned char *__restrict__ codes, int n_relu,
                                   int relu_off) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)batch * ld) return;
    const int b = (int)(idx / ld), t = (int)(idx % ld);
    float ll = 0.0f, lu = 0.0f, nu = 0.0f;
    if (t < n) {
        const float *cs = colsum + (size_t)b * groups_per_box * ld_s;
        float l = 0.0f, u = 0.0f;
        for (int q = 0; q < groups_per_box; ++q) {
            l += cs[(size_t)q * ld_s + t];
            u += cs[(size_t)q * ld_s + n + t];
        }
        CERT_ST(lb_out[(size_t)b * n_total + out_off + t], l);
        CERT_ST(ub_out[(size_t)b * n_total + out_off + t], u);
        if (do_relax) {
            const bool pick_one = (__fadd_rn(l, u) >= 0.0f);   // relu_n
            ll = pick_one ? 1.0f : 0.0f;
            unsigned char code;
            if (l >= 0.0f) {                                    // compute_upper, first test
                lu = 1.0f; code = 1;
            } else if (u <= 0.0f) {                             // second test
                lu = 0.0f; code = 0;
            } else {
                const float den = __fsub_rn(u, l);
                lu = __fdiv_rn(u, den);
                nu = -__fdiv_rn(__fmul_rn(u, l), den);
                code = (unsigned char)(2 + (pick_one ? 1 : 0));
            }
            CERT_ST(codes[(size_t)b * n_relu + relu_off + t], code);
        }
    }
    if (!do_relax) return;
    CERT_ST(lamL[idx], ll);
    CERT_ST(lamU[idx], lu);
    CERT_ST(nuU[idx], nu);
}

// S_k from the raw [L_k | U_k]: L_t *= lamL_t; U_t = lamU_t * U_t, + nuU_t on the constant row (without a ReLU
// the shapes pass unchanged), and S of the first layer from its weights, both written as fp16 pairs
// (x = hi + 2^-11 lo, see gemm_tc16.cuh).
constexpr float kLoScale16 = 2048.0f;

__device__ __forceinline__ void store_pair16(float v, __half &h, __half &l, bool &out_of_range) {
    out_of_range |= !(fabsf(v) <= 60000.0f);
    h = __float2half_rn(v);
    l = __float2half_rn((v - __half2float(h)) * kLoScale16);
}

__device__ __forceinline__ uint4 pack8(const __half (&x)[8]) {
    uint4 p;
    p.x = (uint32_t)__half_as_ushort(x[0]) | ((uint32_t)__half_as_ushort(x[1]) << 16);
    p.y = (uint32_t)__half_as_ushort(x[2]) | ((uint32_t)__half_as_ushort(x[3]) << 16);
    p.z = (uint32_t)__half_as_ushort(x[4]) | ((uint32_t)__half_as_ushort(x[5]) << 16);
    p.w = (uint32_t)__half_as_ushort(x[6]) | ((uint32_t)__half_as_ushort(x[7]) << 16);
    return p;
}

// One warp per row, a lane per group of 8 columns (16-byte stores of halves; pitches are multiples of 32 elements).
__global__ void reuse_init16_kernel(const float *__restrict__ W0t, int ldw, const float *__restrict__ bias,
                                    int n, int n0, int R, int ld_s, int ld_relax, int has_relu,
                                    const float *__restrict__ lamL, const float *__restrict__ lamU,
                                    const float *__restrict__ nuU, long long rows, __half *__restrict__ S_hi,
                                    __half *__restrict__ S_lo, int *__restrict__ status) {
    // one warp per row, lanes over groups of 8 columns
    const int octs = ld_s / 8;
    const long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    bool out_of_range = false;
    const int box = r < rows ? (int)(r / R) : 0, s = r < rows ? (int)(r % R) : 0;
    for (int o = lane; r < rows && o < octs; o += 32) {
        const int col0 = o * 8;
        __half h[8], l[8];
        if ((n & 7) == 0 && (ldw & 3) == 0 && col0 < 2 * n && s <= n0) {
            // the eight columns lie on one side (n a multiple of 8): 16-byte loads of the weights (or the bias on the
            // constant row), the slopes and the intercepts
            const bool upper = col0 >= n;
            const int t0 = upper ? col0 - n : col0;
            const float *base_p = s < n0 ? W0t + (size_t)s * ldw + t0 : bias + t0;
            const float4 b0 = *reinterpret_cast<const float4 *>(base_p), b1 = *reinterpret_cast<const float4 *>(base_p + 4);
            const float base[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            float lam[8] = {1.0f, 1.0f, 1.0f, 1.0f, 1.0f, 1.0f, 1.0f, 1.0f};
            float nu[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
            if (has_relu) {
                const float *lam_p = (upper ? lamU : lamL) + (size_t)box * ld_relax + t0;
                const float4 a0 = *reinterpret_cast<const float4 *>(lam_p), a1 = *reinterpret_cast<const float4 *>(lam_p + 4);
                lam[0] = a0.x; lam[1] = a0.y; lam[2] = a0.z; lam[3] = a0.w; lam[4] = a1.x; lam[5] = a1.y; lam[6] = a1.z; lam[7] = a1.w;
                if (upper && s == n0) {
                    const float *nu_p = nuU + (size_t)box * ld_relax + t0;
                    const float4 n0v = *reinterpret_cast<const float4 *>(nu_p), n1v = *reinterpret_cast<const float4 *>(nu_p + 4);
                    nu[0] = n0v.x; nu[1] = n0v.y; nu[2] = n0v.z; nu[3] = n0v.w; nu[4] = n1v.x; nu[5] = n1v.y; nu[6] = n1v.z; nu[7] = n1v.w;
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) store_pair16(fmaf(lam[e], base[e], nu[e]), h[e], l[e], out_of_range);
            CERT_ST(*reinterpret_cast<uint4 *>(S_hi + (size_t)r * ld_s + col0), pack8(h));
            CERT_ST(*reinterpret_cast<uint4 *>(S_lo + (size_t)r * ld_s + col0), pack8(l));
            continue;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int col = col0 + e;
            float v = 0.0f;
            if (col < 2 * n && s <= n0) {
                const bool upper = col >= n;
                const int t = upper ? col - n : col;
                const float base = s < n0 ? W0t[(size_t)s * ldw + t] : bias[t];
                float lam = 1.0f, nu = 0.0f;
                if (has_relu) {
                    lam = upper ? lamU[(size_t)box * ld_relax + t] : lamL[(size_t)box * ld_relax + t];
                    nu = (upper && s == n0) ? nuU[(size_t)box * ld_relax + t] : 0.0f;
                }
                v = fmaf(lam, base, nu);
            }
            store_pair16(v, h[e], l[e], out_of_range);
        }
        CERT_ST(*reinterpret_cast<uint4 *>(S_hi + (size_t)r * ld_s + col0), pack8(h));
        CERT_ST(*reinterpret_cast<uint4 *>(S_lo + (size_t)r * ld_s + col0), pack8(l));
    }
    if (__any_sync(0xffffffffu, out_of_range) && (threadIdx.x & 31) == 0) atomicOr(status, 2);
}

// raw: fp32 [L_k | U_k] of the contraction; S_hi / S_lo: the scaled shapes as an fp16 pair (other buffers).
__global__ void reuse_scale16_kernel(const float *__restrict__ raw, __half *__restrict__ S_hi,
                                     __half *__restrict__ S_lo, int ld_s, int n, int n0, int R, int ld_relax,
                                     int has_relu, const float *__restrict__ lamL, const float *__restrict__ lamU,
                                     const float *__restrict__ nuU, long long rows, int *__restrict__ status) {
    // one warp per row, lanes over groups of 8 columns
    const int octs = ld_s / 8;
    const long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    bool out_of_range = false;
    const int box = r < rows ? (int)(r / R) : 0, s = r < rows ? (int)(r % R) : 0;
    for (int o = lane; r < rows && o < octs; o += 32) {
        const int col0 = o * 8;
        const float4 r0 = *reinterpret_cast<const float4 *>(raw + (size_t)r * ld_s + col0);
        const float4 r1 = *reinterpret_cast<const float4 *>(raw + (size_t)r * ld_s + col0 + 4);
        const float rv[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
        __half h[8], l[8];
        if ((n & 7) == 0 && col0 < 2 * n && s <= n0 && has_relu) {
            // the eight columns lie on one side (n a multiple of 8): the slopes, and on the constant row the
            // intercepts, come as two 16-byte loads each
            const bool upper = col0 >= n;
            const float *lam_p = (upper ? lamU : lamL) + (size_t)box * ld_relax + (upper ? col0 - n : col0);
            const float4 a0 = *reinterpret_cast<const float4 *>(lam_p), a1 = *reinterpret_cast<const float4 *>(lam_p + 4);
            const float lam[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            float nu[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
            if (upper && s == n0) {
                const float *nu_p = nuU + (size_t)box * ld_relax + (col0 - n);
                const float4 n0v = *reinterpret_cast<const float4 *>(nu_p), n1v = *reinterpret_cast<const float4 *>(nu_p + 4);
                nu[0] = n0v.x; nu[1] = n0v.y; nu[2] = n0v.z; nu[3] = n0v.w;
                nu[4] = n1v.x; nu[5] = n1v.y; nu[6] = n1v.z; nu[7] = n1v.w;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) store_pair16(fmaf(lam[e], rv[e], nu[e]), h[e], l[e], out_of_range);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int col = col0 + e;
                float v = 0.0f;
                if (col < 2 * n && s <= n0) {
                    v = rv[e];
                    if (has_relu) {
                        const bool upper = col >= n;
                        const int t = upper ? col - n : col;
                        const float lam = upper ? lamU[(size_t)box * ld_relax + t] : lamL[(size_t)box * ld_relax + t];
                        const float nu = (upper && s == n0) ? nuU[(size_t)box * ld_relax + t] : 0.0f;
                        v = fmaf(lam, v, nu);
                    }
                }
                store_pair16(v, h[e], l[e], out_of_range);
            }
        }
        CERT_ST(*reinterpret_cast<uint4 *>(S_hi + (size_t)r * ld_s + col0), pack8(h));
        CERT_ST(*reinterpret_cast<uint4 *>(S_lo + (size_t)r * ld_s + col0), pack8(l));
    }
    if (__any_sync(0xffffffffu, out_of_range) && (threadIdx.x & 31) == 0) atomicOr(status, 2);
}

}  // namespace

void launch_reuse_init16(const float *W0t, int ldw, const LayerDev &L0, int n0, int R, int ld_s, long long rows,
                         __half *S_hi, __half *S_lo, int *status, cudaStream_t st) {
    reuse_init16_kernel<<<(unsigned)ceil_div_ll(rows, 8), 256, 0, st>>>(
        W0t, ldw, L0.bias_n, L0.n_out, n0, R, ld_s, L0.ld_out, L0.relu_after, L0.lamL, L0.lamU, L0.nuU, rows, S_hi, S_lo,
        status);
}

void launch_reuse_scale16(const float *raw, __half *S_hi, __half *S_lo, int ld_s, const LayerDev &L, int n0, int R,
                          long long rows, int *status, cudaStream_t st) {
    reuse_scale16_kernel<<<(unsigned)ceil_div_ll(rows, 8), 256, 0, st>>>(
        raw, S_hi, S_lo, ld_s, L.n_out, n0, R, L.ld_out, L.relu_after, L.lamL, L.lamU, L.nuU, rows, status);
}

void launch_reuse_relax(const float *colsum, int ld_s, int groups_per_box, const LayerDev &L, int batch,
                        float *lb_out, float *ub_out, int n_total, unsigned char *codes, int n_relu,
                        cudaStream_t st) {
    const long long threads = (long long)batch * L.ld_out;
    reuse_relax_kernel<<<(unsigned)ceil_div_ll(threads, 256), 256, 0, st>>>(
        colsum, ld_s, groups_per_box, L.n_out, L.ld_out, batch, lb_out, ub_out, n_total, L.out_off, L.relu_after,
        L.lamL, L.lamU, L.nuU, codes, n_relu, L.relu_off);
}

}  // namespace cert
