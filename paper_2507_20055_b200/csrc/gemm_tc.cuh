// Interface of the tensor-core (tcgen05, 3xTF32) affine back-step.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace cert {

constexpr int kTcSmemMax = 227 * 1024;

enum { TC_EPI_RELU = 0, TC_EPI_CONCRETIZE = 1 };

// Storage for a CUtensorMap (128 bytes, 64-byte aligned), kept opaque so that
// only gemm_tc.cu needs the driver API header.
struct alignas(64) TcMap {
    unsigned char bytes[128];
};

struct TcArgs {
    long long M;     // rows of the coefficient matrix = batch * 2 * n_k
    int K;           // neurons of layer j (columns of Q, rows of W_j)
    int n_k;         // neurons of the layer being bounded (decodes a row into box, side, neuron)
    int ld_n;        // padded width of the output (neurons below layer j)
    int bn, bn_pad, n_tiles, stages, tmem_cols;
    int total_tiles; // row panels x column tiles
    int has_relu;    // a ReLU sits on the neurons below layer j
    // ReLU back-step epilogue
    float *out_hi, *out_lo;                      // Q' [M][ld_n]; out_lo == nullptr: unsplit fp32 in out_hi
    const float *lamL, *lamU, *nuU;              // [batch][ld_n]
    const float *bias_below;                     // [ld_n] bias of the affine layer below (next step)
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
    int *status;                                 // set to 1 if a bounded wait runs out
};

bool tc_driver_init();
bool tc_prepare_kernels();
bool tc_make_map(TcMap *m, const float *base, long long inner, long long outer, long long pitch_floats,
                 int box_outer, int bk);
void tc_tile_plan(int N, int bk, int *bn, int *bn_pad, int *n_tiles, int *stages, int *tmem_cols,
                  int *smem_bytes);
void launch_gemm_tc(int epi, int bk, int grid, const TcMap &a_hi, const TcMap &a_lo, const TcMap &b_hi,
                    const TcMap &b_lo, const TcArgs &args, int smem_bytes, cudaStream_t st);

}  // namespace cert
