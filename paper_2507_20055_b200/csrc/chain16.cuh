// Interface of the chain kernel: the whole traversal of an FC layer's expressions in one launch
// (fp16-split tensor-core form, narrow FC nets).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "gemm_tc.cuh"

namespace cert {

constexpr int kChainMaxLayers = 12;     // layers of a net the kernel's parameter block has room for
constexpr int kChainColGroups = 4;     // epilogue warps per TMEM lane quarter = slots a row's bound leaves in
constexpr int kChainMaxWidth = 256;     // neurons of a hidden layer: a 128-row panel of coefficients stays in shared memory

// Layer j as a traversal meets it: the step through it is P = Q * W_j (K = n_out, N = n_in), followed by
// the ReLU back-step through the neurons below it (relaxation of layer j-1) or by the concretisation.
struct ChainLayer {
    int n_out, n_in;
    int ld_in;                          // padded n_in: pitch of the arrays below
    int bn, n_tiles;                    // column tiling of the step through this layer
    int relu_below;                     // a ReLU sits on the neurons below (j >= 1)
    const float *lamL, *lamU, *nuU;     // relaxation of layer j-1, [batch][ld_in]
    const float *bias_below;            // bias of layer j-1, [ld_in]
    float w_unscale;                    // one-pass form: 2^-s, the factor the weight pair of this layer carries, inverted
};

struct ChainParams {
    TcMap b_hi[kChainMaxLayers], b_lo[kChainMaxLayers];   // W_j transposed as an fp16 pair; box = 64 x bn/2
    ChainLayer layer[kChainMaxLayers];
};

struct ChainArgs {
    long long M;                        // rows = 2 * batch * n_k, ordered (box, side, neuron)
    int n_k, k, j_end;                  // the traversal of layer k goes through layers k-1 .. j_end
    const float *Wk;                    // layer k's rows, fp32 [n_k][ldw_k]
    int ldw_k;
    const float *bias_k;
    const float *box_l, *box_u;         // what the result is simplified against, [batch][layer[j_end].ld_in]
    float *d_out;                       // the bound of row r = sum over s < kChainColGroups of d_out[s * slot_stride + r]
    long long slot_stride;
    int *status;                        // bit 0: a bounded wait ran out, bit 1: a coefficient left the fp16 range
    int stages;                         // pipeline stages of W_j tiles
    int a_blocks;                       // 64-column blocks of the coefficient panel held in shared memory
    int b_chunk_bytes;                  // room for one CTA's share of a W_j tile k-block (a multiple of 1024)
    int vec_ld;                         // > 0: the relaxation and bias vectors of a step are staged in shared memory
                                        // (two buffers of 7 * vec_ld floats: bias, then lamL, lamU, nuU of two boxes)
    // One-pass form (see gemm_tc16.cu): the panel holds q_scale * Q (a power of two) as hi + lo with an unscaled lo,
    // the weight maps hold the pairs of 2^s W_j, a k-block of W_j is streamed once for its three products, and the
    // row constants are kept times q_scale until they leave (q_unscale = 1 / q_scale).
    int one_pass;
    float q_scale, q_unscale;
};

bool chain16_prepare();
// Shared memory the kernel needs for `a_blocks`; *stages receives the pipeline depth (< 2: does not fit).
// `max_bnl` = most rows of a W_j tile a CTA stages, `ld_max` = widest padded hidden layer; *vec_ld receives ld_max
// if the staging buffers fit beside three pipeline stages, else 0.
int chain16_smem_bytes(int a_blocks, int max_bnl, int ld_max, int *stages, int *b_chunk_bytes, int *vec_ld);
void launch_chain16(const ChainParams &P, const ChainArgs &a, int pairs, int smem_bytes, cudaStream_t st);

}  // namespace cert
