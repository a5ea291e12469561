// Interface of the tensor-core (tcgen05, 3xTF32) affine back-step.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace cert {

constexpr int kTcSmemMax = 227 * 1024;

// TC_EPI_RELU_SKIP: the ReLU epilogue with the waiting coefficients of a residual connection added first (a
// variant of its own so that the common epilogue carries no code for it).
// TC_EPI_RELU_BAND / TC_EPI_CONCRETIZE_BAND: the two path epilogues for the banded form of a conv back-step
// (TcArgs::n_bands), again as variants of their own.
enum { TC_EPI_RELU = 0, TC_EPI_CONCRETIZE = 1, TC_EPI_REUSE = 2, TC_EPI_RELU_SKIP = 3, TC_EPI_RELU_BAND = 4,
       TC_EPI_CONCRETIZE_BAND = 5, TC_EPI_RELU_BAND_SKIP = 6 };

// Storage for a CUtensorMap (128 bytes, 64-byte aligned), kept opaque so that
// only gemm_tc.cu needs the driver API header.
struct alignas(64) TcMap {
    unsigned char bytes[128];
};

// Tile plan of the back-step through one layer (N = neurons below the layer).
struct TcPlan {
    int bn;          // columns per tile: a multiple of 32, at most 256
    int n_tiles;     // column tiles
    int stages;      // pipeline stages of K
    int tmem_cols;   // tensor-memory columns (two accumulators)
    int smem_bytes;
};

struct TcArgs {
    long long M;     // rows of the coefficient matrix = batch * 2 * n_k
    int K;           // neurons of layer j (columns of Q, rows of W_j)
    int n_k;         // neurons of the layer being bounded (decodes a row into box, side, neuron)
    int ld_n;        // padded width of the output (neurons below layer j)
    int bn, n_tiles, stages, tmem_cols;
    // fp16-split kernel, one-pass form: coefficients travel as pairs of q_scale * Q (q_scale = 2^a, q_unscale = 2^-a);
    // acc_scale = 2^-(a+s) comes off the accumulator (the weights carry 2^s)
    float q_scale, q_unscale, acc_scale;
    int n_narrow;    // fp16-split kernel: the last n_narrow column tiles of a row panel are bn - 32 columns wide
    int total_tiles; // row panels x column tiles (a row panel is 128 rows per CTA of the group)
    // Banded form of a conv back-step on dense coefficient maps (n_bands > 0).  Maps are held row-major by map
    // row ("y-major": [y][channel][x]), so the coefficients of `band_rin` consecutive rows of layer j's output map
    // are one contiguous K window of a row of A, and the `s` rows of the map below that depend on them are one
    // contiguous window of the output row.  A work tile is (row panel, band, column tile of the band); the B
    // operand is the band matrix [s * band_row_out][band_rin * band_row_in], the same for every band.
    //   A window of band i:  rows i - band_o_shift .. + band_rin - 1 of the map, clipped to [0, band_h_in)
    //   output window:       columns (i * band_s - band_y_shift) * band_row_out .. + band_s * band_row_out - 1,
    //                        32-column chunks outside [0, ld_n) are dropped
    // The relaxation / box arrays are y-major copies, indexed by the output column.
    int n_bands, band_rin, band_o_shift, band_h_in, band_row_in;   // band_row_in = channels * width of layer j's output map
    int band_s, band_y_shift, band_row_out;                        // band_row_out = channels * width of the map below
    int band_c_out, band_h_out, band_w_out;                        // the map below, for add_identity: the row's own neuron
                                                                   // (channel-major index row mod n_k) sits at its y-major column
    int has_relu;    // a ReLU sits on the neurons below layer j
    int split_out;   // ReLU epilogue: store the result as a TF32 pair (a tensor-core step follows)
    const float *lamL, *lamU, *nuU;              // [batch][ld_n] ("box" = whatever a group of 2 * n_k rows shares)
    const float *bias_below;                     // [ld_n] bias of the affine layer below (next step)
    // ReLU epilogue, residual connection ending on the neurons below layer j: coefficients added to the
    // product before the ReLU back-step: a matrix [rows][ld_n] (fp32, or a TF32 pair), and / or the unit
    // coefficient of the row's own neuron (column = row mod n_k).  (The fp16-split kernel reads the two
    // pointers as the hi and lo halves of an fp16 pair; both are then set.)
    const float *add_hi, *add_lo;
    int add_identity;
    // concretisation epilogue
    const float *l0, *u0;                        // [batch][ld_n]
    // Row constants travel in slots: the constant of row r so far is the sum over
    // s < n_slots_in of d_in[s*slot_stride + r]; this launch writes n_tiles slots to d_out
    // (slot 0 includes the sum of the input slots).  For the concretising epilogue the
    // output slots sum to the bound itself.  Fixed order, no atomics.
    const float *d_in;
    float *d_out;
    int n_slots_in;
    long long slot_stride;
    // TC_EPI_REUSE (fp16-split kernel only; shapes kept over the input layer): a row is (box, s) with s < reuse_n0 an input
    // coordinate, s == reuse_n0 the constant, rows per box = reuse_R (a multiple of 32); a column is a
    // neuron's lower (col < n_half) or upper (n_half <= col < 2*n_half) shape.  The result is stored
    // unsplit; bias2[col] is added on the constant row; colsum[(row / 32) * ld_n + col] receives the sum
    // over the warp's 32 rows of the column's concretisation terms against the box l0, u0 [box][reuse_ld0].
    int reuse_R, reuse_n0, reuse_ld0, n_half;
    const float *bias2;
    float *colsum;
    int *status;                                 // set to 1 if a bounded wait runs out
    const int *run_if;                           // not null: the launch has no work tiles unless *run_if != 0 when it starts
};

// One block that waits, with a short limit, on a barrier nothing arrives on, and then raises bit 0 of *status.
void launch_bounded_wait_selftest(int *status, cudaStream_t st);
bool tc_driver_init();
// Sets the kernels' shared-memory limits; *pair_ok tells whether the two-CTA form can be launched.
bool tc_prepare_kernels(bool *pair_ok);
// 2D fp32 tensor [outer][inner] with row pitch `pitch_floats`; box = 32 floats x box_outer rows, 128-byte swizzle.
bool tc_make_map(TcMap *m, const float *base, long long inner, long long outer, long long pitch_floats,
                 int box_outer);
TcPlan tc_tile_plan(int N, int ctas);
// ctas = 1: one CTA per 128-row panel; ctas = 2: a CTA pair shares a 256-row panel (cta_group::2).
// `groups` = CTAs (ctas = 1) or CTA pairs (ctas = 2) to launch.
void launch_gemm_tc(int epi, int ctas, int groups, const TcMap &a_hi, const TcMap &a_lo, const TcMap &b_hi,
                    const TcMap &b_lo, const TcMap &o_hi, const TcMap &o_lo, const TcArgs &args, int smem_bytes,
                    cudaStream_t st);

}  // namespace cert
