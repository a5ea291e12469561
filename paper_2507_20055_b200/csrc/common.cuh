// Shared declarations of the library's translation units (device structs,
// launch wrappers, error helpers).  Notation follows the paper: an affine
// layer k computes z_k = W_k a_{k-1} + b_k; `curr` neurons index rows of W_k,
// `prev` neurons its columns (Section 3.2).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cstdint>
#include <cstdio>
#include <utility>
#include "../../include/cert.h"

namespace cert {

constexpr int kPad = 32;  // every row of a coefficient / weight / relaxation array is padded to 32 floats

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// Programmatic dependent launch for the chain of small dependent kernels of a call: a kernel lets the next one
// be scheduled as soon as all of its own blocks have started (pdl_trigger), and touches global memory only
// after the kernel before it has completed and flushed (pdl_wait).  Launch latency and each kernel's
// set-up (barriers, tensor memory) then overlap the tail of the kernel before.  Both are no-ops for a kernel
// launched without the attribute.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
bool pdl_enabled();   // false when the environment variable CERT_PDL is 0

template <typename Kernel, typename... Args>
inline void launch_chained(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
inline long long ceil_div_ll(long long a, long long b) { return (a + b - 1) / b; }

// ---- checked stores (a build with -DCERT_BOUNDS; memory-safety evidence, not for production) ----
// Every plain store to global memory in the kernels that do not go through TMA is written CERT_ST(lvalue, value).
// In an ordinary build that is the assignment.  In a CERT_BOUNDS build the address is first looked up in a table of
// the buffers the current call may write (the net's allocations and the caller's output arrays, uploaded before
// the call's first launch); a store that falls outside every one of them is skipped and raises bit 2 of the
// table's status word (cert_net_last_status then returns CERT_ERR_BOUNDS).  Nothing faults either way.
#ifdef CERT_BOUNDS
constexpr int kBoundsMax = 1024;
struct BoundsTable {
    int n;
    int *status;
    unsigned long long lo[kBoundsMax], hi[kBoundsMax];
};
// Host side: each translation unit with kernels keeps its own device copy of the table (no relocatable device
// code is used) and registers an uploader for it when the library is loaded.
void bounds_register_uploader(void (*upload)(const BoundsTable *));
void bounds_upload_all(const BoundsTable *t);      // synchronises the device, then calls every uploader
#ifdef __CUDACC__
static __device__ BoundsTable g_bounds_table;
__device__ __forceinline__ bool bounds_check(const void *p, size_t bytes) {
    const unsigned long long a = (unsigned long long)p;
    for (int i = 0; i < g_bounds_table.n; ++i)
        if (a >= g_bounds_table.lo[i] && a + bytes <= g_bounds_table.hi[i]) return true;
    if (g_bounds_table.status) atomicOr(g_bounds_table.status, 4);
    return false;
}
namespace {
inline void bounds_upload_this_unit(const BoundsTable *t) { cudaMemcpyToSymbol(g_bounds_table, t, sizeof(BoundsTable)); }
struct BoundsRegistrar {
    BoundsRegistrar() { bounds_register_uploader(&bounds_upload_this_unit); }
};
static BoundsRegistrar g_bounds_registrar;
}  // namespace
#define CERT_ST(lvalue, value)                                                        \
    do {                                                                              \
        if (cert::bounds_check(&(lvalue), sizeof(lvalue))) (lvalue) = (value);        \
    } while (0)
#endif
#else
#define CERT_ST(lvalue, value) ((lvalue) = (value))
#endif

// One affine layer on the device.
struct LayerDev {
    int kind, relu_after;
    int n_in, n_out;         // neurons below / of this layer
    int ld_in, ld_out;       // padded to kPad
    int c_in, h_in, w_in, c_out, kh, kw, stride, pad, h_out, w_out;
    float *W;                // FC: [round_up(n_out,kPad)][ld_in], zero padded.  CONV: [c_out][c_in][kh][kw]
    float *Wt_hi, *Wt_lo;    // FC only: TF32 split of W transposed, [round_up(n_in,kPad)][ld_out] (rows = prev neuron)
    float *Wct;              // CONV only: [c_out][kh][kw][c_in] (c_in innermost) for the transposed-conv kernel
    float *bias_n;           // [ld_out] one bias per neuron (conv: per-channel bias expanded), zero padded
    int out_off;             // offset of this layer's neurons in lb_out / ub_out rows
    int relu_off;            // offset in the branch-code rows (valid if relu_after)
    // relaxation of the ReLU on top (valid if relu_after): [max_batch][ld_out]
    float *lamL, *lamU, *nuU;
    // concrete bounds of this layer's outputs (after its ReLU, if any): [max_batch][ld_out]; null for the last layer
    float *actL, *actU;
};

// Conv geometry handed to kernels by value.
struct ConvGeom {
    int c_in, h_in, w_in, c_out, kh, kw, stride, pad, h_out, w_out;
};

inline ConvGeom geom_of(const LayerDev &L) {
    return ConvGeom{L.c_in, L.h_in, L.w_in, L.c_out, L.kh, L.kw, L.stride, L.pad, L.h_out, L.w_out};
}

// ---- launch wrappers (each enqueues exactly one kernel on `st`) ----

#ifdef CERT_BOUNDS
// Attempts CERT_ST(p[0], 1): with p outside every registered buffer the store is skipped and the status bit raised.
void launch_checked_store_selftest(float *p, cudaStream_t st);
#endif
// *out = max(*out, max |x[i]|) for *out >= 0 (set-up time: the range proof of the fp16 split).
void launch_absmax(const float *x, long long n, float *out, cudaStream_t st);

// l0 = max(c - eps, lo), u0 = min(c + eps, hi); rows padded with zeros.
void launch_box(const float *centers, float eps, float lo, float hi, int batch, int n0, int ld0,
                float *l0, float *u0, cudaStream_t st);

// Bounds of an affine layer without traversal: simplify_lower/upper of the layer's rows against
// the concrete bounds l0, u0 [batch][ld0] of its inputs (the box for the first layer, where the
// expression is already over the input; the bounds of the layer below for an interval step).
void launch_first_layer_bounds(const LayerDev &L, const float *l0, const float *u0, int ld0, int batch,
                               float *lb_out, float *ub_out, int n_total, cudaStream_t st);

// Relu transformer: relaxation (lamL, lamU, nuU) and branch code from (l, u).
// With `slots` != nullptr the bounds are first summed from n_slots partial sums per row
// (rows ordered (box, side, neuron), slot s at slots + s*slot_stride) and stored to lb_out / ub_out;
// the relaxation itself is skipped for a layer without a ReLU.
// slot_npos > 0: the slot rows are ordered (box, position, side, channel) for a conv layer with slot_npos
// output positions (the order of the tensor-core patch steps) instead of (box, side, neuron).
void launch_relax(const LayerDev &L, float *lb_out, float *ub_out, int n_total, int batch,
                  unsigned char *codes, int n_relu, const float *slots, int n_slots, long long slot_stride,
                  cudaStream_t st, int slot_npos = 0, const int *run_if = nullptr);

// Start of the back-substitution for layer k: the expression of neuron i is
// row i of W_k (the same for every box and both sides) and the constant b_k[i];
// it is pushed through the ReLU below (if any) right away, and the constant
// picks up Q.b of the affine layer below, through which the next step goes.
//   Q  [rows][ld] with rows = batch*2*n_k ordered (box, side, neuron)
//   Q_lo != nullptr: Q is written as a TF32 pair (hi in Q, lo in Q_lo) for the tensor-core contraction
// run_if != nullptr (here, in launch_relax and in TcArgs, FC layers): the kernel does its work only if *run_if is
// non-zero when it starts; it belongs to a re-run that an earlier kernel of the same call may have made necessary.
void launch_init_expr(const LayerDev &Lk, const LayerDev &Lbelow, int batch, float *Q, float *Q_lo, float *d,
                      cudaStream_t st, int y_major = 0,    // y_major (conv layer k): columns in [y][channel][x] order
                      const int *run_if = nullptr);

// ReLU back-step in place on P [rows][ld] (expression over the outputs of
// layer `Lj`, i.e. over its ReLU neurons if it has one), plus d += Q.b_j.
// The row constant comes in as the sum of n_slots slots of d and leaves in slot 0.
void launch_relu_step(const LayerDev &Lj, int batch, int n_k, float *P, float *P_lo, float *d, int n_slots,
                      long long slot_stride, cudaStream_t st);

// P [rows][ld] += the waiting coefficients of a residual connection (see ConvtEpilogue::add_hi): S_hi (+ S_lo),
// or 1 at column (row mod n_k) when `identity`.
void launch_add_skip(float *P, const float *S_hi, const float *S_lo, int identity, long long rows, int n, int ld,
                     int n_k, cudaStream_t st);

// Interval step of layer Lk with a residual connection from layer Ls: lb += actL_s, ub += actU_s.
void launch_add_act_bounds(const LayerDev &Lk, const LayerDev &Ls, int batch, float *lb_out, float *ub_out,
                           int n_total, cudaStream_t st);
// A traversal of layer Lk's rows stopped while coefficients (S_hi (+ S_lo) [rows][Ls.ld_out], and / or the unit
// coefficient of the row's own neuron) still waited on layer Ls's outputs: their simplification against Ls's
// concrete output bounds goes to `slot` [rows] if given, else is added to lb_out / ub_out.
void launch_skip_concretize(const float *S_hi, const float *S_lo, int identity, const LayerDev &Ls, long long rows,
                            const LayerDev &Lk, float *slot, float *lb_out, float *ub_out, int n_total,
                            cudaStream_t st);

// map(simplify_lower/upper): rows of P [rows][ld0] against the box.
void launch_concretize(const float *P, const float *d, int n_slots, long long slot_stride, const float *l0,
                       const float *u0, int n0, int ld0, int batch, int n_k, float *lb_out, float *ub_out, int n_total, int out_off,
                       cudaStream_t st);

// C[M][ldc] = A[M][lda] * B[K][ldb]  (fp32 FMA units).  Columns up to ldc are
// written (B is zero padded), so padded outputs are zero.
void launch_gemm_ffma(const float *A, int lda, const float *B, int ldb, float *C, int ldc, long long M,
                      int N, int K, cudaStream_t st);

// What the conv back-step kernel applies to its result while it is still in registers.
enum { CONVT_EPI_RELU = 0, CONVT_EPI_CONCRETIZE = 1 };
struct ConvtEpilogue {
    int mode;                 // CONVT_EPI_RELU: ReLU back-step through the layer below + constant's share of the
                              // next affine step, result stored; CONVT_EPI_CONCRETIZE: bounds against the box
    int n_k;                  // neurons of the layer being bounded (decodes a row into box, side, neuron)
    // row constants: sum over n_slots_in slots of d_in in, slot 0 of d_out out (may be the same buffer)
    const float *d_in;
    int n_slots_in;
    long long slot_stride;
    float *d_out;
    // CONVT_EPI_RELU
    int has_relu;
    const float *lamL, *lamU, *nuU;   // [batch][ld_in] relaxation of the ReLU below
    const float *bias_below;          // [ld_in]
    float *P, *P_lo;                  // result [rows][ld_in]; P_lo != nullptr: stored as a TF32 pair
    // Residual connection ending on the neurons below: coefficients that waited for the traversal to reach
    // them are added before the ReLU back-step: a matrix [rows][ld_in] (fp32, or a TF32 pair), or the unit
    // coefficient of the row's own neuron (the layer being bounded has the connection itself).
    const float *add_hi, *add_lo;
    int add_identity;
    // CONVT_EPI_CONCRETIZE
    const float *l0, *u0;             // [batch][ld_in]
    float *lb_out, *ub_out;
    int n_total, out_off;
};

// P[r][(ci,iy,ix)] = sum over (co,ky,kx) of Q[r][(co,oy,ox)] * W[co][ci][ky][kx]: the exact
// transpose of the conv layer applied to every row's coefficient map, followed by `ep`.
// `sms`: number of multiprocessors (the kernel is persistent).
void launch_convt_ffma(const LayerDev &L, const float *Q, long long rows, int sms, const ConvtEpilogue &ep,
                       cudaStream_t st);

// ---- conv back-steps on receptive-field patches (conv_patch.cu) ----
// One level of a conv neuron's expression held as a window [c][ph][pw] whose origin in the map is
// (oy, ox) * a - b for the neuron's output position (oy, ox).
struct PatchLevel {
    int c, ph, pw, a, b, elems, pitch;
};
// Plans the traversal of conv layer k's expressions through layers k-1 .. j_end on patches:
// levels[0] is over the outputs of layer k-1, levels[m] over the inputs of layer k-m.  False when a
// layer on the way is not a conv layer or a window is not much smaller than its map.
bool conv_patch_plan(const LayerDev *layers, int k, int j_end, PatchLevel *levels, int max_levels);
void conv_patch_prepare();
// Start: the kernel of layer k as a patch over the outputs of the layer below, through that layer's ReLU.
// `pitch` floats per row; patch_lo != nullptr: written as a TF32 pair for a tensor-core step, with the rows
// ordered (box, position, side, channel) so that the rows of a tile share their position-dependent vectors.
void launch_patch_start(const LayerDev &Lk, const LayerDev &Lb, int pitch, int batch, float *patch,
                        float *patch_lo, float *d, cudaStream_t st);
// For the tensor-core form of a patch back-step (the conv layer as a dense matrix between windows, the
// same for every position): windows of n_arr <= 3 per-neuron arrays [batch][Lj.ld_in] of the layer below
// conv layer j, one vector of ld_dst floats per (box, output position of layer k), zero outside the map;
// a null src[i] stands for fill[i] inside the map.
void launch_patch_gather(const LayerDev &Lk, const LayerDev &Lj, const PatchLevel &out, int ld_dst, int batch,
                         int n_arr, const float *const *src, const float *fill, float *const *dst,
                         cudaStream_t st);
// Back-step of the patches through conv layer j, followed by `ep` (ep.P = output patches, pitch out.pitch).
void launch_patch_step(const LayerDev &Lk, const LayerDev &Lj, const PatchLevel &in, const PatchLevel &out,
                       const float *in_patch, long long rows, int sms, const ConvtEpilogue &ep, cudaStream_t st);

// ---- y-major copies for the banded tensor-core form of the dense conv back-steps (conv_patch.cu) ----
// Maps [c][h][w] -> [h][c][w]: a coefficient matrix held as a TF32 pair, and up to three per-neuron arrays
// [batch][ld] (a null src[i] stands for fill[i]).
void launch_to_ymajor_pair(const float *src_hi, const float *src_lo, float *dst_hi, float *dst_lo, long long rows,
                           int c, int h, int w, int ld, cudaStream_t st);
void launch_to_ymajor_vectors(int c, int h, int w, int ld, int batch, int n_arr, const float *const *src,
                              const float *fill, float *const *dst, cudaStream_t st);

// ---- ReuseCert (reuse.cu): shapes over the input layer, one matrix S per layer ----
// S rows are (box, s): s < n0 input coordinate, s == n0 constant, zero rows up to R per box; columns
// [L (n) | U (n)] padded to ld_s.  S is held as an fp16 pair (x = hi + 2^-11 lo); `status` bit 1 is raised when
// a value leaves the fp16 range.
// Bounds (and the relaxation, under a ReLU) of layer L from the contraction's column sums.
void launch_reuse_relax(const float *colsum, int ld_s, int groups_per_box, const LayerDev &L, int batch,
                        float *lb_out, float *ub_out, int n_total, unsigned char *codes, int n_relu,
                        cudaStream_t st);
// The first layer's S, and the scale step (reads the raw fp32 result from one buffer, writes the pair to others).
void launch_reuse_init16(const float *W0t, int ldw, const LayerDev &L0, int n0, int R, int ld_s, long long rows,
                         __half *S_hi, __half *S_lo, int *status, cudaStream_t st);
void launch_reuse_scale16(const float *raw, __half *S_hi, __half *S_lo, int ld_s, const LayerDev &L, int n0, int R,
                          long long rows, int *status, cudaStream_t st);
}  // namespace cert
