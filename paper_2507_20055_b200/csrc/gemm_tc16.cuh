// Interface of the fp16-split tensor-core affine back-step (CERT_CONTRACTION_TC3XFP16).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cstdint>

#include "gemm_tc.cuh"

namespace cert {

// An fp32 value x is held as hi = fp16(x) and lo = fp16(2^11 * (x - hi)): 22 bits of significand, as the
// TF32 pair, at half the bytes and twice the tensor-core rate.  Products are exact in the fp32
// accumulator; the cross terms (in units of 2^-11) are accumulated first and scaled by 2^-11 on the way
// into the hi*hi pass.  Range: |x| must stay below 65504 (a larger coefficient raises the range flag,
// bit 1 of the status word); below 6.1e-5 the pair is exact to 1.5e-11 absolute.
// The one-pass form holds 2^a x as hi = fp16(2^a x), lo = fp16(2^a x - hi): the same 22 bits while
// |2^a x| >= 2^-3 (below that lo is a subnormal, exact to 2^-25 absolute), and |2^a x| must stay below 65504.
constexpr float kLoScale = 2048.0f;

struct Tc16Plan {
    int bn, n_tiles, stages, tmem_cols, smem_bytes;
    int n_narrow;    // the last n_narrow column tiles are bn - 32 wide (N = 784: 224 + 3 x 192 instead of 4 x 224)
};

bool tc16_prepare_kernels();
// 2D fp16 tensor [outer][inner], row pitch in elements; box = box_inner x box_outer elements;
// box_inner = 64 -> 128-byte swizzle (operand tiles), 32 -> 64-byte swizzle (epilogue slabs).
bool tc16_make_map(TcMap *m, const __half *base, long long inner, long long outer, long long pitch_elems,
                   int box_inner, int box_outer);
// n_tiles = 0: as few column tiles as 256 columns per tile allow; n_tiles > 0: that many (launches with too few row
// panels to give every CTA pair a 256-column tile take more, narrower ones)
Tc16Plan tc16_tile_plan(int N, int n_tiles = 0);
// CTA pairs only.  TcArgs as for the TF32 kernel; d_out receives 2 * n_tiles slots per row.
// one_pass == false: both operands are pairs (fp16(x), fp16(2^11 (x - hi))), two passes over K.
// one_pass == true (not for TC_EPI_REUSE): both operands are pairs with unscaled lo parts of 2^a Q and 2^s W
// (TcArgs::q_scale = 2^a, q_unscale = 2^-a, acc_scale = 2^-(a+s)); a k-block is staged once for its three products.
void launch_gemm_tc16(int epi, bool one_pass, int pairs, const TcMap &a_hi, const TcMap &a_lo, const TcMap &b_hi,
                      const TcMap &b_lo, const TcMap &o_hi, const TcMap &o_lo, const TcArgs &args, int smem_bytes,
                      cudaStream_t st);
// Start of a traversal at FC layer k as an fp16 pair (see launch_init_expr): hi = fp16(q_scale x),
// lo = fp16(lo_scale (q_scale x - hi)).
struct LayerDev;
void launch_init_expr16(const LayerDev &Lk, const LayerDev &Lbelow, int batch, __half *Q_hi, __half *Q_lo, float *d,
                        int *status, float q_scale, float lo_scale, cudaStream_t st);

}  // namespace cert
