// Affine back-step C' = C * W_j on the fp32 FMA units (Section 4.3, Matmul
// rewrite: the traversal step over an affine layer is a matrix product).
// Plain shared-memory tiled SGEMM, 128x128x8 tiles, 8x8 outputs per thread.
// Fallback and cross-check for the tensor-core path.
#include "common.cuh"

namespace cert {

namespace {

constexpr int BM = 128, BN = 128, BK = 8;

// A [M][lda] row-major with zero-padded columns up to a multiple of kPad,
// B [>= round_up(K,kPad)][ldb] row-major zero padded, C [M][ldc]; ldb == ldc.
__global__ void __launch_bounds__(256)
sgemm_nn_kernel(const float *__restrict__ A, int lda, const float *__restrict__ B, int ldb,
                float *__restrict__ C, int ldc, long long M, int K) {
    __shared__ __align__(16) float As[2][BK][BM];
    __shared__ __align__(16) float Bs[2][BK][BN];
    const int tid = threadIdx.x;
    // one-dimensional grid (row tile major): the y extent of a grid stops at 65535 tiles, rows do not
    const int col_tiles = (ldc + BN - 1) / BN;
    const long long row0 = (long long)(blockIdx.x / col_tiles) * BM;
    const int col0 = (int)(blockIdx.x % col_tiles) * BN;
    const int ty = tid / 16, tx = tid % 16;

    // global -> register staging
    const int a_row = tid / 2, a_k = (tid % 2) * 4;
    const int b_k = tid / 32, b_col = (tid % 32) * 4;
    const bool a_ok = (row0 + a_row) < M;
    const bool b_ok = (col0 + b_col) < ldb;
    const float *a_ptr = A + (size_t)(row0 + a_row) * lda + a_k;
    const float *b_ptr = B + (size_t)b_k * ldb + col0 + b_col;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    const int k_tiles = (K + BK - 1) / BK;   // K is padded with zeros up to a multiple of kPad
    float4 a_reg = a_ok ? *reinterpret_cast<const float4 *>(a_ptr) : make_float4(0, 0, 0, 0);
    float4 b_reg = b_ok ? *reinterpret_cast<const float4 *>(b_ptr) : make_float4(0, 0, 0, 0);
    int buf = 0;
    As[buf][a_k + 0][a_row] = a_reg.x; As[buf][a_k + 1][a_row] = a_reg.y;
    As[buf][a_k + 2][a_row] = a_reg.z; As[buf][a_k + 3][a_row] = a_reg.w;
    *reinterpret_cast<float4 *>(&Bs[buf][b_k][b_col]) = b_reg;
    __syncthreads();

    for (int kt = 0; kt < k_tiles; ++kt) {
        if (kt + 1 < k_tiles) {
            a_reg = a_ok ? *reinterpret_cast<const float4 *>(a_ptr + (size_t)(kt + 1) * BK) : make_float4(0, 0, 0, 0);
            b_reg = b_ok ? *reinterpret_cast<const float4 *>(b_ptr + (size_t)(kt + 1) * BK * ldb) : make_float4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float4 a0 = *reinterpret_cast<const float4 *>(&As[buf][k][ty * 4]);
            float4 a1 = *reinterpret_cast<const float4 *>(&As[buf][k][64 + ty * 4]);
            float4 b0 = *reinterpret_cast<const float4 *>(&Bs[buf][k][tx * 4]);
            float4 b1 = *reinterpret_cast<const float4 *>(&Bs[buf][k][64 + tx * 4]);
            float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (kt + 1 < k_tiles) {
            buf ^= 1;
            As[buf][a_k + 0][a_row] = a_reg.x; As[buf][a_k + 1][a_row] = a_reg.y;
            As[buf][a_k + 2][a_row] = a_reg.z; As[buf][a_k + 3][a_row] = a_reg.w;
            *reinterpret_cast<float4 *>(&Bs[buf][b_k][b_col]) = b_reg;
            __syncthreads();
        }
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        long long row = row0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (row >= M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int col = col0 + (h == 0 ? tx * 4 : 64 + tx * 4);
            if (col < ldc)
                CERT_ST(*reinterpret_cast<float4 *>(&C[(size_t)row * ldc + col]),
                        make_float4(acc[i][h * 4 + 0], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]));
        }
    }
}

}  // namespace

void launch_gemm_ffma(const float *A, int lda, const float *B, int ldb, float *C, int ldc, long long M, int N,
                      int K, cudaStream_t st) {
    (void)N;
    const long long col_tiles = (ldc + BN - 1) / BN;
    long long row_tiles_left = ceil_div_ll(M, BM);
    const long long max_row_tiles = 0x7FFFFFFFLL / col_tiles;      // blocks of one launch: at most 2^31 - 1
    long long row0 = 0;
    while (row_tiles_left > 0) {
        const long long t = row_tiles_left < max_row_tiles ? row_tiles_left : max_row_tiles;
        const long long rows = (M - row0) < t * BM ? (M - row0) : t * BM;
        sgemm_nn_kernel<<<(unsigned)(t * col_tiles), 256, 0, st>>>(A + row0 * lda, lda, B, ldb, C + row0 * ldc, ldc,
                                                                 rows, K);
        row_tiles_left -= t;
        row0 += t * BM;
    }
}

}  // namespace cert
