// C ABI of the library: network object, workspace, and the per-call schedule
// of kernel launches that realises the DeepPoly flow (Appendix C, DeepPoly
// listing): flow(forward) over layers; at each affine layer a traversal
// backward through every earlier layer; concretisation at the input; then
// the Relu transformer picks the relaxation used by later traversals.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc16.cuh"
#include "chain16.cuh"

// Tensor-core operands of the back-step through one FC layer j: B = W_j transposed
// (rows = neurons below, K-major), A = the coefficient matrix over layer j's neurons
// in either ping-pong buffer.
// The same operands for the fp16-split kernel (CTA pairs only).
struct Tc16Layer {
    bool usable = false;
    __half *W_hi = nullptr, *W_lo = nullptr;     // W_j transposed, [round_up(n_in, 32)][ld_out]
    cert::TcMap b_hi, b_lo, a_hi[3], a_lo[3], o_hi[3], o_lo[3];   // one per coefficient buffer
    cert::Tc16Plan plan;
    // One-pass form: W' = 2^w_shift W_j as Wh = fp16(W'), Wl = fp16(W' - Wh), same layout.  w_shift puts the
    // largest |W'| in [2^14, 2^15), so Wl is a normal fp16 number wherever |W| >= 2^-18 max|W|.
    bool one_pass = false;
    __half *Ws_hi = nullptr, *Ws_lo = nullptr;
    cert::TcMap s_hi, s_lo;
    float w_unscale = 1.0f;                      // 2^-w_shift
    // More, narrower column tiles for launches whose row panels are too few to give every CTA pair a 256-column
    // tile (small batches, the output layer's traversal): finer[i] has plan.n_tiles + 1 + i column tiles (up to
    // kMaxFineTiles) and weight maps with the matching box; the output maps are the common ones.
    struct Finer { cert::Tc16Plan plan; cert::TcMap hi, lo; bool ok = false; };
    std::vector<Finer> finer;
};
constexpr int kMaxFineTiles = 16;

struct TcLayer {
    bool usable = false;
    cert::TcMap b_hi, b_lo;          // box = this CTA's share of the column tile
    cert::TcMap a_hi[3], a_lo[3];    // one per coefficient buffer
    cert::TcMap o_hi[3], o_lo[3];    // store maps of the result (width = neurons below, padded); j >= 1 only
    cert::TcPlan plan;
};


// Tensor-core form of one patch back-step: the rows of conv layer k, held as windows over the outputs of
// conv layer j (level m = k-1-j), go to windows over j's inputs.  Between windows the conv layer is one
// dense matrix T [K = c_out*ph*pw][N = c_in*qh*qw], the same for every neuron position and box, so the
// step is a plain contraction; what depends on the position (the relaxation or the box at the window's
// place in the map, and which window positions lie outside the map) enters through per-(box, position)
// vectors gathered before the launch.
struct TcPatchStep {
    int K = 0, Kp = 0, N = 0, ldN = 0;   // window elements in / out and their padded widths
    float *T_hi = nullptr, *T_lo = nullptr;      // T transposed, [ldN][Kp], TF32 split
    float *bias_e = nullptr;             // [ldN] bias of the affine layer below, per window element; null at j = 0
    cert::TcMap b_hi, b_lo, a_hi[2], a_lo[2], o_hi[2], o_lo[2];
    cert::TcPlan plan;
};

// Banded tensor-core form of the back-step through conv layer j on dense coefficient maps (TcArgs::n_bands):
// s consecutive rows of the map below depend on `rin` consecutive rows of layer j's output map only, and the
// matrix between the two is the same for every band.  With the maps held y-major both windows are contiguous
// pieces of a row, so the step is the ordinary contraction with a K window per tile.  Usable for layer j when it
// is for every layer below too: a traversal, once its matrix is y-major, stays on this form to its end.
struct BandStep {
    bool usable = false;
    int K = 0, N = 0;                    // rin * c_out * w_out; s * c_in * w_in (both multiples of 32)
    int rin = 0, o_shift = 0, y_shift = 0, n_bands = 0;
    float *T_hi = nullptr, *T_lo = nullptr;      // band matrix transposed, [N][K], TF32 split
    float *bias_y = nullptr;             // [ld_in] bias of layer j-1 per neuron, y-major; null for j = 0
    float *bias_out_y = nullptr;         // [ld_out] this layer's bias per output neuron, y-major
    float *W_above_y = nullptr;          // the FC layer j+1's weights with their columns in y-major order, [pad(n)][ld_out]
                                         // (a traversal that starts there writes its first matrix y-major at once)
    cert::TcMap b_hi, b_lo, a_hi[3], a_lo[3], o_hi[3], o_lo[3];   // one per coefficient buffer
    cert::TcPlan plan;
};

// ReuseCert (served in the fp16 split): per affine layer k >= 1 the block weight matrix
// [[W+^T, W-^T], [W-^T, W+^T]] as the K-major B operand (rows = the 2*n_k output columns, columns = the 2*n_{k-1}
// columns of the layer below) as an fp16 pair; the shapes rotate through three buffers (pair in, raw fp32
// result, pair out).
struct ReuseLayer {
    int ld_s = 0;                        // pitch of this layer's [L | U] matrix
    float *bias2 = nullptr;
    __half *B16_hi = nullptr, *B16_lo = nullptr;
    cert::TcMap b16_hi, b16_lo, a16_hi[3], a16_lo[3], o32[3];
    cert::Tc16Plan plan16;
};

struct ReuseState {
    bool on = false;
    int R = 0;                           // rows per box: n0 coordinates, the constant, zero padding to 32
    float *W0t = nullptr;                // first layer's weights transposed [round_up(n0, 32)][ld_out]
    float *X[3] = {nullptr, nullptr, nullptr};   // shape buffers: an fp16 pair (hi, then lo at lo_off halves) or a raw fp32 result
    size_t lo_off = 0;
    float *colsum = nullptr;
    std::vector<ReuseLayer> layers;
};

struct cert_net {
    int n_layers = 0, max_batch = 0;
    float clip_lo = 0, clip_hi = 0;
    int n0 = 0, ld0 = 0, n_total = 0, n_relu = 0;
    int device = 0;
    int contraction = CERT_CONTRACTION_AUTO;
    std::vector<cert::LayerDev> layers;
    std::vector<void *> allocs;   // every device allocation, for destroy
    // Guard words: every allocation is kGuardBytes longer at either end, filled with kGuardByte at create;
    // cert_net_check_guards reads them back (a kernel that writes beyond a buffer lands there first).
    struct Guarded { unsigned char *base; size_t bytes; };
    std::vector<Guarded> guards;
    float *l0 = nullptr, *u0 = nullptr;      // [max_batch][ld0]
    // coefficient matrices (fp32, or the TF32 hi parts): two that alternate, and for nets with residual
    // connections a third, so that the matrix a connection sets aside stays put while the traversal goes on
    float *buf[3] = {nullptr, nullptr, nullptr};
    float *buf_lo[3] = {nullptr, nullptr, nullptr};   // TF32 lo parts for the tensor-core contraction
    float *zeros = nullptr;                  // [widest layer, padded] zeros (nets with residual connections)
    std::vector<int> skip_from;              // residual connections: layer k adds the outputs of layer skip_from[k] (-1: none); empty: none at all
    int n_buf = 2;
    bool tc_ok = false;                      // tensor-core path usable on this net
    std::vector<TcLayer> tc;                 // per layer: operand maps and tile plan
    bool tc16_ok = false;                    // fp16-split path usable (FC layers only, CTA pairs available)
    bool tc16_one_pass = false;              // its layers all have the operands of the one-pass form
    // AUTO takes the fp16 split: the net's weights prove that no coefficient of any traversal can leave the
    // fp16 range (fp16_coef_bound = the largest entry of |W_k| |W_k-1| ... |W_j| over all k > j >= 1; slopes of a
    // ReLU back-step lie in [0, 1], so every stored coefficient is below it in magnitude)
    // AUTO, layers whose proof fails (deep nets): the traversal runs in the fp16 split all the same, reporting to a
    // status word of its own (spec_dev[k], cleared at the start of a call), and is followed by the same traversal
    // in the TF32 split whose kernels do nothing unless that word came up (an overflow, or a run-out wait).
    bool speculate = false;
    int *spec_dev = nullptr;                 // [n_layers]
    bool auto_fp16 = false;                  // some layer's traversal passes the proof
    float fp16_coef_bound = INFINITY;        // the largest bound over all layers
    std::vector<float> fp16_layer_bound;     // [k]: the bound for the traversal of layer k (k >= 1)
    std::vector<Tc16Layer> tc16;
    // fp16-split path, narrow nets: a whole traversal per launch with the coefficient panel kept in shared memory
    bool chain_ok = false;
    cert::ChainParams chain;
    int chain_a_blocks = 0, chain_stages = 0, chain_smem = 0, chain_chunk = 0, chain_vec_ld = 0;
    float *dbuf[2] = {nullptr, nullptr};     // row constants, [d_slots][slot_stride] each, ping-pong
    int d_slots = 1;                         // slots per buffer (most column tiles of any contraction)
    long long slot_stride = 0;               // rows of the largest coefficient matrix
    int sm_count = 148;
    int tc_ctas = 1;                         // CTAs per row panel of the tensor-core kernel (2: cta_group::2)
    bool conv_patches = true;                // conv-sourced rows travel as receptive-field patches where they can
    std::vector<std::vector<TcPatchStep>> tcp;   // [k]: the leading patch steps of layer k's traversal that can run on the tensor cores
    float *gat[3] = {nullptr, nullptr, nullptr}; // gathered windows, [max_batch * positions][ldN] each (y-major vectors for the banded form)
    size_t gat_floats = 0;
    std::vector<BandStep> band;                  // [j]: banded tensor-core form of the step through conv layer j
    bool band_residual_ok = true;                // every layer a residual connection ends on takes the banded form
    ReuseState reuse;
    unsigned char *codes = nullptr;          // [max_batch][n_relu]
    int *status_dev = nullptr;               // sticky device status word
    // host staging for cert_deeppoly_bounds_host
    float *centers_dev = nullptr, *lb_dev = nullptr, *ub_dev = nullptr;
    int last_batch = 0;
    int last_launches = 0;
    int last_paths = 0;              // bit 0: an FFMA contraction ran, bit 1: a tensor-core one, bit 2: in CTA pairs, bit 3: a traversal ran on patches
    // optional per-launch event timing (events are created when profiling is switched on)
    bool profiling = false;
    std::vector<cudaEvent_t> prof_events;
    std::vector<int> prof_class;   // class of the launch between event i and i+1
    int prof_marks = 0;
};

constexpr int kMaxPatchLevels = 16;

#ifdef CERT_BOUNDS
namespace { std::vector<void (*)(const cert::BoundsTable *)> &bounds_uploaders(); }
namespace cert {
void bounds_register_uploader(void (*upload)(const BoundsTable *)) { bounds_uploaders().push_back(upload); }
void bounds_upload_all(const BoundsTable *t) {
    cudaDeviceSynchronize();
    for (auto fn : bounds_uploaders()) fn(t);
}
}  // namespace cert
#endif

namespace cert {
bool convt_supported(const LayerDev &L);
void convt_prepare();
}  // namespace cert

namespace {

using cert::LayerDev;
using cert::kPad;
using cert::round_up;

constexpr size_t kGuardBytes = 256;        // keeps the payload 256-byte aligned
constexpr int kGuardByte = 0xA5;

bool dev_alloc(cert_net *net, void **p, size_t bytes) {
    if (bytes == 0) bytes = 256;
    unsigned char *base = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&base), bytes + 2 * kGuardBytes) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return false;
    }
    net->allocs.push_back(base);
    if (cudaMemset(base, kGuardByte, kGuardBytes) != cudaSuccess ||
        cudaMemset(base + kGuardBytes + bytes, kGuardByte, kGuardBytes) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return false;
    }
    net->guards.push_back({base, bytes});
    *p = base + kGuardBytes;
    return true;
}

template <typename T>
bool dev_alloc_zero(cert_net *net, T **p, size_t count) {
    if (!dev_alloc(net, reinterpret_cast<void **>(p), count * sizeof(T))) return false;
    return cudaMemset(*p, 0, (count ? count : 1) * sizeof(T)) == cudaSuccess;
}

void free_net(cert_net *net) {
    if (!net) return;
    for (cudaEvent_t e : net->prof_events) cudaEventDestroy(e);
    for (void *p : net->allocs) cudaFree(p);
    delete net;
}

// Neurons of a (validated) conv layer descriptor.
int desc_conv_out(const cert_layer_desc_t &L) {
    const int ho = (L.h_in + 2 * L.pad - L.kh) / L.stride + 1, wo = (L.w_in + 2 * L.pad - L.kw) / L.stride + 1;
    return L.c_out * ho * wo;
}

cert_status_t validate(const cert_layer_desc_t *layers, int n_layers, int max_batch, float clip_lo,
                       float clip_hi) {
    if (!layers || n_layers < 1 || max_batch < 1) return CERT_ERR_INVALID_ARG;
    if (std::isnan(clip_lo) || std::isnan(clip_hi) || clip_lo > clip_hi) return CERT_ERR_INVALID_ARG;
    long long prev_out = -1;
    for (int k = 0; k < n_layers; ++k) {
        const cert_layer_desc_t &L = layers[k];
        if (!L.weight || !L.bias) return CERT_ERR_INVALID_ARG;
        if (L.relu_after != 0 && L.relu_after != 1) return CERT_ERR_INVALID_ARG;
        long long n_in, n_out;
        if (L.kind == CERT_LAYER_FC) {
            if (L.in_features < 1 || L.out_features < 1) return CERT_ERR_INVALID_ARG;
            n_in = L.in_features;
            n_out = L.out_features;
        } else if (L.kind == CERT_LAYER_CONV2D) {
            if (L.c_in < 1 || L.h_in < 1 || L.w_in < 1 || L.c_out < 1 || L.kh < 1 || L.kw < 1 ||
                L.stride < 1 || L.pad < 0)
                return CERT_ERR_INVALID_ARG;
            if (L.h_in + 2 * L.pad < L.kh || L.w_in + 2 * L.pad < L.kw) return CERT_ERR_INVALID_ARG;
            int ho = (L.h_in + 2 * L.pad - L.kh) / L.stride + 1, wo = (L.w_in + 2 * L.pad - L.kw) / L.stride + 1;
            n_in = (long long)L.c_in * L.h_in * L.w_in;
            n_out = (long long)L.c_out * ho * wo;
        } else {
            return CERT_ERR_INVALID_ARG;
        }
        if (n_in > (1 << 20) || n_out > (1 << 20)) return CERT_ERR_UNSUPPORTED;
        if (prev_out >= 0 && n_in != prev_out) return CERT_ERR_INVALID_ARG;
        prev_out = n_out;
    }
    return CERT_OK;
}

// TF32 with round-to-nearest, ties away from zero (what cvt.rna.tf32.f32 does), for finite inputs.
float host_tf32(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    u = (u + 0x1000u) & 0xFFFFE000u;
    float r;
    std::memcpy(&r, &u, 4);
    return r;
}

// Uploads the TF32 split of every FC layer's transposed weights and encodes the TMA
// descriptors.  Failure to reach the driver entry point leaves the FFMA path in use.
cert_status_t setup_tensor_core_path(cert_net *net, const cert_layer_desc_t *descs, size_t max_elems) {
    const int K = net->n_layers;
    net->tc.assign(K, TcLayer());
    net->tc_ok = false;
    if (K < 2) return CERT_OK;
    bool pair_ok = false;
    if (!cert::tc_driver_init() || !cert::tc_prepare_kernels(&pair_ok)) return CERT_OK;
    net->tc_ctas = (pair_ok && net->sm_count >= 2) ? 2 : 1;
    if (const char *e = std::getenv("CERT_TC_CTAS")) {
        if (std::atoi(e) == 1) net->tc_ctas = 1;
    }
    const int ctas = net->tc_ctas;
    for (int p = 0; p < net->n_buf; ++p)
        if (!dev_alloc_zero(net, &net->buf_lo[p], max_elems)) return CERT_ERR_OOM;
    std::vector<float> hi, lo;
    for (int j = 0; j < K - 1; ++j) {
        LayerDev &L = net->layers[j];
        if (L.kind != CERT_LAYER_FC) continue;
        TcLayer &T = net->tc[j];
        // W_j transposed: row s (neuron below), column t (neuron of layer j), pitch ld_out
        size_t rows_pad = round_up(L.n_in, kPad);
        hi.assign(rows_pad * L.ld_out, 0.0f);
        lo.assign(rows_pad * L.ld_out, 0.0f);
        for (int t = 0; t < L.n_out; ++t)
            for (int s2 = 0; s2 < L.n_in; ++s2) {
                float w = descs[j].weight[(size_t)t * L.n_in + s2];
                float h = host_tf32(w);
                hi[(size_t)s2 * L.ld_out + t] = h;
                lo[(size_t)s2 * L.ld_out + t] = host_tf32(w - h);
            }
        if (!dev_alloc(net, (void **)&L.Wt_hi, hi.size() * sizeof(float)) ||
            !dev_alloc(net, (void **)&L.Wt_lo, lo.size() * sizeof(float)))
            return CERT_ERR_OOM;
        if (cudaMemcpy(L.Wt_hi, hi.data(), hi.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(L.Wt_lo, lo.data(), lo.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
            return CERT_ERR_CUDA;
        T.plan = cert::tc_tile_plan(L.n_in, ctas);
        if (T.plan.stages < 2) continue;
        bool ok = cert::tc_make_map(&T.b_hi, L.Wt_hi, L.n_out, L.n_in, L.ld_out, T.plan.bn / ctas) &&
                  cert::tc_make_map(&T.b_lo, L.Wt_lo, L.n_out, L.n_in, L.ld_out, T.plan.bn / ctas);
        // rows of the largest layer above j
        long long rows_max = 0;
        for (int k = j + 1; k < K; ++k) rows_max = std::max(rows_max, 2LL * net->max_batch * net->layers[k].n_out);
        for (int p = 0; p < net->n_buf && ok; ++p) {
            ok = cert::tc_make_map(&T.a_hi[p], net->buf[p], L.n_out, rows_max, L.ld_out, 128) &&
                 cert::tc_make_map(&T.a_lo[p], net->buf_lo[p], L.n_out, rows_max, L.ld_out, 128);
            if (ok && j > 0)
                ok = cert::tc_make_map(&T.o_hi[p], net->buf[p], L.ld_in, rows_max, L.ld_in, 32) &&
                     cert::tc_make_map(&T.o_lo[p], net->buf_lo[p], L.ld_in, rows_max, L.ld_in, 32);
        }
        T.usable = ok;
        if (ok) net->d_slots = std::max(net->d_slots, T.plan.n_tiles);
    }
    net->tc_ok = true;

    // fp16-split operands: nets of FC layers, CTA pairs available
    bool all_fc = true;
    for (int j = 0; j < K; ++j) all_fc = all_fc && net->layers[j].kind == CERT_LAYER_FC;
    net->tc16.assign(K, Tc16Layer());
    if (all_fc && ctas == 2 && cert::tc16_prepare_kernels()) {
        bool all_ok = true, all_one_pass = true;
        std::vector<__half> h16, l16;
        bool one_pass_wanted = true;
        if (const char *e = std::getenv("CERT_TC16_ONE_PASS")) one_pass_wanted = std::atoi(e) != 0;
        for (int j = 0; j < K - 1 && all_ok; ++j) {
            LayerDev &L = net->layers[j];
            Tc16Layer &T = net->tc16[j];
            size_t rows_pad = round_up(L.n_in, kPad);
            h16.assign(rows_pad * L.ld_out, __float2half_rn(0.0f));
            l16.assign(rows_pad * L.ld_out, __float2half_rn(0.0f));
            for (int t = 0; t < L.n_out; ++t)
                for (int s2 = 0; s2 < L.n_in; ++s2) {
                    const float w = descs[j].weight[(size_t)t * L.n_in + s2];
                    if (!(std::fabs(w) <= 60000.0f)) all_ok = false;
                    const __half h = __float2half_rn(w);
                    h16[(size_t)s2 * L.ld_out + t] = h;
                    l16[(size_t)s2 * L.ld_out + t] = __float2half_rn((w - __half2float(h)) * cert::kLoScale);
                }
            if (!dev_alloc(net, (void **)&T.W_hi, h16.size() * sizeof(__half)) ||
                !dev_alloc(net, (void **)&T.W_lo, l16.size() * sizeof(__half)))
                return CERT_ERR_OOM;
            if (cudaMemcpy(T.W_hi, h16.data(), h16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess ||
                cudaMemcpy(T.W_lo, l16.data(), l16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess)
                return CERT_ERR_CUDA;
            T.plan = cert::tc16_tile_plan(L.n_in);
            if (T.plan.stages < 2) { all_ok = false; break; }
            bool ok = cert::tc16_make_map(&T.b_hi, T.W_hi, L.n_out, L.n_in, L.ld_out, 64, T.plan.bn / 2) &&
                      cert::tc16_make_map(&T.b_lo, T.W_lo, L.n_out, L.n_in, L.ld_out, 64, T.plan.bn / 2);
            if (ok && all_ok && one_pass_wanted) {
                float wmax = 0.0f;
                for (size_t i = 0; i < (size_t)L.n_out * L.n_in; ++i) wmax = std::max(wmax, std::fabs(descs[j].weight[i]));
                int e = 0;
                if (wmax > 0.0f) std::frexp(wmax, &e);               // wmax = m 2^e, m in [0.5, 1)
                const int shift = wmax > 0.0f ? std::min(std::max(15 - e, -24), 24) : 0;
                const float up = std::ldexp(1.0f, shift);
                std::fill(h16.begin(), h16.end(), __float2half_rn(0.0f));
                std::fill(l16.begin(), l16.end(), __float2half_rn(0.0f));
                for (int t = 0; t < L.n_out; ++t)
                    for (int s2 = 0; s2 < L.n_in; ++s2) {
                        const float w = descs[j].weight[(size_t)t * L.n_in + s2] * up;   // exact
                        const __half h = __float2half_rn(w);
                        h16[(size_t)s2 * L.ld_out + t] = h;
                        l16[(size_t)s2 * L.ld_out + t] = __float2half_rn(w - __half2float(h));
                    }
                if (!dev_alloc(net, (void **)&T.Ws_hi, h16.size() * sizeof(__half)) ||
                    !dev_alloc(net, (void **)&T.Ws_lo, l16.size() * sizeof(__half)))
                    return CERT_ERR_OOM;
                if (cudaMemcpy(T.Ws_hi, h16.data(), h16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess ||
                    cudaMemcpy(T.Ws_lo, l16.data(), l16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess)
                    return CERT_ERR_CUDA;
                T.w_unscale = std::ldexp(1.0f, -shift);
                T.one_pass = cert::tc16_make_map(&T.s_hi, T.Ws_hi, L.n_out, L.n_in, L.ld_out, 64, T.plan.bn / 2) &&
                             cert::tc16_make_map(&T.s_lo, T.Ws_lo, L.n_out, L.n_in, L.ld_out, 64, T.plan.bn / 2);
                const int units = (L.n_in + 31) / 32;
                for (int nt = T.plan.n_tiles + 1; T.one_pass && nt <= std::min(units, kMaxFineTiles); ++nt) {
                    Tc16Layer::Finer F;
                    F.plan = cert::tc16_tile_plan(L.n_in, nt);
                    F.ok = F.plan.stages >= 2 &&
                           cert::tc16_make_map(&F.hi, T.Ws_hi, L.n_out, L.n_in, L.ld_out, 64, F.plan.bn / 2) &&
                           cert::tc16_make_map(&F.lo, T.Ws_lo, L.n_out, L.n_in, L.ld_out, 64, F.plan.bn / 2);
                    if (F.ok) net->d_slots = std::max(net->d_slots, 2 * nt);
                    T.finer.push_back(F);
                }
            }
            all_one_pass = all_one_pass && T.one_pass;
            long long rows_max = 0;
            for (int k = j + 1; k < K; ++k) rows_max = std::max(rows_max, 2LL * net->max_batch * net->layers[k].n_out);
            for (int p = 0; p < net->n_buf && ok; ++p) {
                const __half *bh = reinterpret_cast<const __half *>(net->buf[p]);
                const __half *bl = reinterpret_cast<const __half *>(net->buf_lo[p]);
                ok = cert::tc16_make_map(&T.a_hi[p], bh, L.n_out, rows_max, L.ld_out, 64, 128) &&
                     cert::tc16_make_map(&T.a_lo[p], bl, L.n_out, rows_max, L.ld_out, 64, 128);
                if (ok && j > 0)
                    ok = cert::tc16_make_map(&T.o_hi[p], bh, L.ld_in, rows_max, L.ld_in, 32, 32) &&
                         cert::tc16_make_map(&T.o_lo[p], bl, L.ld_in, rows_max, L.ld_in, 32, 32);
            }
            T.usable = ok;
            all_ok = all_ok && ok;
            if (ok) net->d_slots = std::max(net->d_slots, 2 * T.plan.n_tiles);
        }
        net->tc16_ok = all_ok;
        net->tc16_one_pass = all_ok && all_one_pass;
        // The chain kernel: every layer a traversal passes through at most kChainMaxWidth neurons wide.
        bool chain = all_ok && net->skip_from.empty() && K <= cert::kChainMaxLayers && cert::chain16_prepare();
        if (const char *e = std::getenv("CERT_CHAIN")) chain = chain && std::atoi(e) != 0;
        int widest = 0;
        for (int j = 0; j + 1 < K; ++j) widest = std::max(widest, net->layers[j].n_out);
        if (chain && widest <= cert::kChainMaxWidth) {
            net->chain_a_blocks = (widest + 63) / 64;
            int max_bnl = 0;
            for (int j = 0; j + 1 < K; ++j) max_bnl = std::max(max_bnl, net->tc16[j].plan.bn / 2);
            net->chain_smem = cert::chain16_smem_bytes(net->chain_a_blocks, max_bnl, round_up(widest, kPad),
                                                       &net->chain_stages, &net->chain_chunk, &net->chain_vec_ld);
            std::memset(&net->chain, 0, sizeof(net->chain));
            for (int j = 0; j < K; ++j) {
                const LayerDev &L = net->layers[j];
                cert::ChainLayer &C = net->chain.layer[j];
                C.n_out = L.n_out; C.n_in = L.n_in; C.ld_in = L.ld_in;
                if (j + 1 < K) {
                    // (the one-pass form's pairs of the scaled weights where the net has them)
                    net->chain.b_hi[j] = net->tc16_one_pass ? net->tc16[j].s_hi : net->tc16[j].b_hi;
                    net->chain.b_lo[j] = net->tc16_one_pass ? net->tc16[j].s_lo : net->tc16[j].b_lo;
                    C.w_unscale = net->tc16[j].w_unscale;
                    C.bn = net->tc16[j].plan.bn; C.n_tiles = net->tc16[j].plan.n_tiles;
                }
                if (j > 0) {
                    const LayerDev &Lb = net->layers[j - 1];
                    C.relu_below = Lb.relu_after;
                    C.lamL = Lb.lamL; C.lamU = Lb.lamU; C.nuU = Lb.nuU; C.bias_below = Lb.bias_n;
                }
            }
            net->chain_ok = net->chain_stages >= 2;
            net->d_slots = std::max(net->d_slots, cert::kChainColGroups);
        }
    }
    return CERT_OK;
}

// Range proof for the fp16 split (FC nets without residual connections).  A traversal of layer k holds, over the
// outputs of layer j-1, the matrix W_k D W_{k-1} D ... W_j with diagonal ReLU slopes D in [0, 1] (sign-split
// scaling never enlarges a coefficient), so each of its entries is at most the matching entry of
// |W_k| |W_{k-1}| ... |W_j| in magnitude.  Those products are formed here, once, on the FMA units (the row
// count is n_k, not batch * 2 * n_k); their largest entry, per layer k, goes to net->fp16_layer_bound[k].  Below
// kFp16Safe the fp16 split cannot overflow in that layer's traversal, whatever the input boxes, and AUTO takes
// it for that layer (the products grow with the number of layers a traversal passes, so on deep nets the first
// layers pass and the last ones stay on the TF32 split).
#ifdef CERT_BOUNDS
cert_status_t bounds_sync(cert_net *net, const void *const *extra, const size_t *extra_bytes, int n_extra);
#endif
constexpr int kQaMax = 14, kQaTrial = 4;     // exponents of the one-pass fp16 form's coefficient scale (run_tc16_steps)
constexpr float kFp16Safe = 60000.0f;       // fp16's largest finite value is 65504; the margin covers fp32 rounding here

cert_status_t prove_fp16_range(cert_net *net) {
    const int K = net->n_layers;
    net->auto_fp16 = false;
    net->fp16_coef_bound = INFINITY;
    net->fp16_layer_bound.assign(K, INFINITY);
    if (!net->tc16_ok) return CERT_OK;
    if (!net->skip_from.empty()) {
        // residual connections add waiting coefficients to a traversal's matrix, which the products below do not
        // cover: no layer is proven, every full traversal runs in the fp16 split on trial (see cert_net::speculate)
        bool all_tc = net->tc_ok;
        for (int j = 0; j + 1 < K; ++j) all_tc = all_tc && net->tc[j].usable;
        bool on = all_tc;
        if (const char *e = std::getenv("CERT_AUTO_FP16")) on = on && std::atoi(e) != 0;
        if (const char *e = std::getenv("CERT_SPECULATE_FP16")) on = on && std::atoi(e) != 0;
        net->speculate = on;
        if (on && !dev_alloc_zero(net, &net->spec_dev, (size_t)K)) return CERT_ERR_OOM;
        return CERT_OK;
    }
#ifdef CERT_BOUNDS
    {
        const cert_status_t bs = bounds_sync(net, nullptr, nullptr, 0);     // the products go through the checked FMA kernel
        if (bs != CERT_OK) return bs;
    }
#endif
    std::vector<float *> absW(K, nullptr);
    float *max_dev = nullptr;
    cert_status_t rc = CERT_OK;
    auto cleanup = [&]() {
        for (float *p : absW) if (p) cudaFree(p);
        if (max_dev) cudaFree(max_dev);
    };
    if (cudaMalloc(reinterpret_cast<void **>(&max_dev), K * sizeof(float)) != cudaSuccess ||
        cudaMemset(max_dev, 0, K * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_OOM;
    }
    std::vector<float> host;
    for (int j = 0; j < K && rc == CERT_OK; ++j) {
        const LayerDev &L = net->layers[j];
        const size_t n = (size_t)round_up(L.n_out, kPad) * L.ld_in;
        host.resize(n);
        if (cudaMemcpy(host.data(), L.W, n * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = CERT_ERR_CUDA; break; }
        for (float &v : host) v = std::fabs(v);
        if (cudaMalloc(reinterpret_cast<void **>(&absW[j]), n * sizeof(float)) != cudaSuccess) { rc = CERT_ERR_OOM; break; }
        if (cudaMemcpy(absW[j], host.data(), n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) rc = CERT_ERR_CUDA;
    }
    for (int k = 1; k < K && rc == CERT_OK; ++k) {
        const LayerDev &Lk = net->layers[k];
        // the start of the traversal: |W_k| itself, rows padded like the coefficient matrices
        const float *cur = absW[k];
        cert::launch_absmax(cur, (long long)Lk.n_out * Lk.ld_in, max_dev + k, nullptr);
        int p = 0;
        for (int j = k - 1; j >= 1; --j) {
            const LayerDev &Lj = net->layers[j];
            cert::launch_gemm_ffma(cur, Lj.ld_out, absW[j], Lj.ld_in, net->buf[p], Lj.ld_in, Lk.n_out, Lj.n_in, Lj.n_out,
                                   nullptr);
            cert::launch_absmax(net->buf[p], (long long)Lk.n_out * Lj.ld_in, max_dev + k, nullptr);
            cur = net->buf[p];
            p ^= 1;
        }
    }
    std::vector<float> bound(K, INFINITY);
    if (rc == CERT_OK &&
        (cudaDeviceSynchronize() != cudaSuccess ||
         cudaMemcpy(bound.data(), max_dev, K * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess))
        rc = CERT_ERR_CUDA;
    // the products went through the coefficient buffers: leave them as the kernels expect to find them (zero)
    if (rc == CERT_OK && K > 2) {
        size_t used = 0;
        for (int k = 1; k < K; ++k)
            for (int j = 1; j < k; ++j) used = std::max(used, (size_t)net->layers[k].n_out * net->layers[j].ld_in);
        for (int p = 0; p < 2; ++p)
            if (cudaMemset(net->buf[p], 0, used * sizeof(float)) != cudaSuccess) rc = CERT_ERR_CUDA;
    }
    cleanup();
    if (rc != CERT_OK) { cudaGetLastError(); return rc; }
    bool off = false;
    if (const char *e = std::getenv("CERT_AUTO_FP16")) off = std::atoi(e) == 0;
    net->fp16_coef_bound = 0.0f;
    for (int k = 1; k < K; ++k) {
        net->fp16_layer_bound[k] = bound[k];
        net->fp16_coef_bound = std::max(net->fp16_coef_bound, bound[k]);
        if (!off && std::isfinite(bound[k]) && bound[k] <= kFp16Safe) net->auto_fp16 = true;
    }
    if (off) net->fp16_layer_bound.assign(K, INFINITY);
    // speculation needs every re-run kernel to be one that takes the predicate: FC steps on the tensor cores
    bool all_tc = net->tc_ok;
    for (int j = 0; j + 1 < K; ++j) all_tc = all_tc && net->tc[j].usable;
    net->speculate = !off && all_tc;
    if (const char *e = std::getenv("CERT_SPECULATE_FP16")) net->speculate = net->speculate && std::atoi(e) != 0;
    if (net->speculate && !dev_alloc_zero(net, &net->spec_dev, (size_t)K)) return CERT_ERR_OOM;
    return CERT_OK;
}

// Patch back-steps on the tensor cores: builds, for every conv layer k over conv layers, the dense
// window-to-window matrices of the leading steps of its traversal.  A step qualifies while the dense
// form does at most kPatchDenseRatio times the multiply-adds of the transposed convolution itself
// (the tensor cores are far more than that ahead of the FMA patch kernel) and the matrix stays small.
constexpr int kPatchDenseRatio = 24;
constexpr size_t kPatchMatrixMax = 16u << 20;   // floats

cert_status_t setup_patch_tc(cert_net *net, const cert_layer_desc_t *descs) {
    const int K = net->n_layers;
    net->tcp.assign(K, std::vector<TcPatchStep>());
    if (!net->tc_ok || !net->skip_from.empty()) return CERT_OK;
    const int ctas = net->tc_ctas;
    size_t gat_floats = 0;
    std::vector<float> hi, lo, be;
    for (int k = 1; k < K; ++k) {
        const LayerDev &Lk = net->layers[k];
        if (Lk.kind != CERT_LAYER_CONV2D) continue;
        cert::PatchLevel lv[kMaxPatchLevels];
        int j_end = 0;
        while (j_end < k && !cert::conv_patch_plan(net->layers.data(), k, j_end, lv, kMaxPatchLevels)) ++j_end;
        if (j_end >= k) continue;
        const long long rows_max = 2LL * net->max_batch * Lk.n_out;
        for (int j = k - 1, m = 0; j >= j_end; --j, ++m) {
            const LayerDev &Lj = net->layers[j];
            const cert::PatchLevel &in = lv[m], &out = lv[m + 1];
            TcPatchStep S;
            S.K = in.elems; S.Kp = round_up(in.elems, kPad);
            S.N = out.elems; S.ldN = round_up(out.elems, kPad);
            if (out.ph * out.pw > kPatchDenseRatio * Lj.kh * Lj.kw) break;
            if ((size_t)S.ldN * S.Kp > kPatchMatrixMax) break;
            S.plan = cert::tc_tile_plan(S.N, ctas);
            if (S.plan.stages < 2) break;
            hi.assign((size_t)S.ldN * S.Kp, 0.0f);
            lo.assign((size_t)S.ldN * S.Kp, 0.0f);
            const float *W = descs[j].weight;          // [c_out][c_in][kh][kw]
            for (int co = 0; co < Lj.c_out; ++co)
                for (int py = 0; py < in.ph; ++py)
                    for (int px = 0; px < in.pw; ++px) {
                        const size_t kk = ((size_t)co * in.ph + py) * in.pw + px;
                        for (int ci = 0; ci < Lj.c_in; ++ci)
                            for (int ky = 0; ky < Lj.kh; ++ky)
                                for (int kx = 0; kx < Lj.kw; ++kx) {
                                    const size_t n = ((size_t)ci * out.ph + Lj.stride * py + ky) * out.pw +
                                                     Lj.stride * px + kx;
                                    const float w = W[(((size_t)co * Lj.c_in + ci) * Lj.kh + ky) * Lj.kw + kx];
                                    const float h = host_tf32(w);
                                    hi[n * S.Kp + kk] = h;
                                    lo[n * S.Kp + kk] = host_tf32(w - h);
                                }
                    }
            if (!dev_alloc(net, (void **)&S.T_hi, hi.size() * sizeof(float)) ||
                !dev_alloc(net, (void **)&S.T_lo, lo.size() * sizeof(float)))
                return CERT_ERR_OOM;
            if (cudaMemcpy(S.T_hi, hi.data(), hi.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess ||
                cudaMemcpy(S.T_lo, lo.data(), lo.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                return CERT_ERR_CUDA;
            if (j > 0 && net->layers[j - 1].kind == CERT_LAYER_CONV2D) {
                // a window element of channel c meets the bias of channel c of the conv layer below
                be.assign(S.ldN, 0.0f);
                const int qhw = out.ph * out.pw;
                for (int e = 0; e < S.N; ++e) be[e] = descs[j - 1].bias[e / qhw];
                if (!dev_alloc(net, (void **)&S.bias_e, be.size() * sizeof(float))) return CERT_ERR_OOM;
                if (cudaMemcpy(S.bias_e, be.data(), be.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                    return CERT_ERR_CUDA;
            }
            bool ok = cert::tc_make_map(&S.b_hi, S.T_hi, S.Kp, S.ldN, S.Kp, S.plan.bn / ctas) &&
                      cert::tc_make_map(&S.b_lo, S.T_lo, S.Kp, S.ldN, S.Kp, S.plan.bn / ctas);
            for (int p = 0; p < 2 && ok; ++p)
                ok = cert::tc_make_map(&S.a_hi[p], net->buf[p], S.Kp, rows_max, S.Kp, 128) &&
                     cert::tc_make_map(&S.a_lo[p], net->buf_lo[p], S.Kp, rows_max, S.Kp, 128) &&
                     cert::tc_make_map(&S.o_hi[p], net->buf[p], S.ldN, rows_max, S.ldN, 32) &&
                     cert::tc_make_map(&S.o_lo[p], net->buf_lo[p], S.ldN, rows_max, S.ldN, 32);
            if (!ok) break;
            net->d_slots = std::max(net->d_slots, S.plan.n_tiles);
            gat_floats = std::max(gat_floats, (size_t)net->max_batch * Lk.h_out * Lk.w_out * S.ldN);
            net->tcp[k].push_back(S);
        }
    }
    net->gat_floats = std::max(net->gat_floats, gat_floats);
    return CERT_OK;
}

// Banded form of the dense conv back-steps, from the first layer upward while map rows are whole k-blocks
// (channels * width a multiple of 32 on both sides) and the dense band matrix does at most kBandDenseRatio
// times the multiply-adds of the convolution itself (the split contraction runs about twenty times the rate the
// FMA kernels reach on these steps; 3 x 3 stride-2 first layers on 3-channel inputs come to 15).
constexpr int kBandDenseRatio = 16;

cert_status_t setup_band_tc(cert_net *net, const cert_layer_desc_t *descs) {
    const int K = net->n_layers;
    net->band.assign(K, BandStep());
    if (!net->tc_ok) return CERT_OK;
    if (const char *e = std::getenv("CERT_CONV_BANDS")) {
        if (std::atoi(e) == 0) return CERT_OK;
    }
    const int ctas = net->tc_ctas;
    std::vector<float> hi, lo, be;
    for (int j = 0; j + 1 < K; ++j) {
        const LayerDev &L = net->layers[j];
        if (L.kind != CERT_LAYER_CONV2D) break;
        BandStep S;
        const int s = L.stride;
        const int row_in = L.c_out * L.w_out, row_out = L.c_in * L.w_in;
        if (row_in % 32 || row_out % 32) break;
        // rows of the output map a band needs: oy' = o_shift + (dy + pad - y_shift - ky) / s over all (dy, ky)
        int best_rin = 1 << 30;
        for (int ys = 0; ys < s; ++ys) {
            int qmin = 1 << 30, qmax = -(1 << 30);
            for (int dy = 0; dy < s; ++dy)
                for (int ky = 0; ky < L.kh; ++ky) {
                    const int num = dy + L.pad - ys - ky;
                    if (((num % s) + s) % s) continue;
                    const int q = num >= 0 ? num / s : -((-num) / s);
                    qmin = std::min(qmin, q); qmax = std::max(qmax, q);
                }
            if (qmax >= qmin && qmax - qmin + 1 < best_rin) {
                best_rin = qmax - qmin + 1; S.rin = best_rin; S.o_shift = -qmin; S.y_shift = ys;
            }
        }
        if (best_rin > 8) break;
        S.K = S.rin * row_in;
        S.N = s * row_out;
        S.n_bands = (L.h_in + S.y_shift + s - 1) / s;
        // every band must reach at least one row of the map (its accumulator is written by its first k-block)
        bool reach = true;
        for (int i = 0; i < S.n_bands; ++i)
            reach = reach && (i - S.o_shift < L.h_out) && (i - S.o_shift + S.rin > 0);
        if (!reach) break;
        if ((long long)S.K * S.N * S.n_bands > (long long)kBandDenseRatio * L.n_out * L.c_in * L.kh * L.kw) break;
        if ((size_t)S.K * S.N > (size_t)(16u << 20)) break;
        S.plan = cert::tc_tile_plan(S.N, ctas);
        if (S.plan.stages < 2) break;
        hi.assign((size_t)S.N * S.K, 0.0f);
        lo.assign((size_t)S.N * S.K, 0.0f);
        const float *W = descs[j].weight;
        for (int dy = 0; dy < s; ++dy)
            for (int ci = 0; ci < L.c_in; ++ci)
                for (int ix = 0; ix < L.w_in; ++ix) {
                    const size_t n = ((size_t)dy * L.c_in + ci) * L.w_in + ix;
                    for (int r = 0; r < S.rin; ++r) {
                        const int ky = dy + L.pad - S.y_shift + s * (S.o_shift - r);
                        if (ky < 0 || ky >= L.kh) continue;
                        for (int co = 0; co < L.c_out; ++co)
                            for (int ox = 0; ox < L.w_out; ++ox) {
                                const int kx = ix + L.pad - s * ox;
                                if (kx < 0 || kx >= L.kw) continue;
                                const size_t kk = ((size_t)r * L.c_out + co) * L.w_out + ox;
                                const float w = W[(((size_t)co * L.c_in + ci) * L.kh + ky) * L.kw + kx];
                                const float h = host_tf32(w);
                                hi[n * S.K + kk] = h;
                                lo[n * S.K + kk] = host_tf32(w - h);
                            }
                    }
                }
        if (!dev_alloc(net, (void **)&S.T_hi, hi.size() * sizeof(float)) ||
            !dev_alloc(net, (void **)&S.T_lo, lo.size() * sizeof(float)))
            return CERT_ERR_OOM;
        if (cudaMemcpy(S.T_hi, hi.data(), hi.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(S.T_lo, lo.data(), lo.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
            return CERT_ERR_CUDA;
        if (j > 0) {
            be.assign(L.ld_in, 0.0f);
            for (int y = 0; y < L.h_in; ++y)
                for (int ci = 0; ci < L.c_in; ++ci)
                    for (int x = 0; x < L.w_in; ++x) be[((size_t)y * L.c_in + ci) * L.w_in + x] = descs[j - 1].bias[ci];
            if (!dev_alloc(net, (void **)&S.bias_y, be.size() * sizeof(float))) return CERT_ERR_OOM;
            if (cudaMemcpy(S.bias_y, be.data(), be.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                return CERT_ERR_CUDA;
        }
        long long rows_max = 0;
        for (int k = j + 1; k < K; ++k) rows_max = std::max(rows_max, 2LL * net->max_batch * net->layers[k].n_out);
        bool ok = cert::tc_make_map(&S.b_hi, S.T_hi, S.K, S.N, S.K, S.plan.bn / ctas) &&
                  cert::tc_make_map(&S.b_lo, S.T_lo, S.K, S.N, S.K, S.plan.bn / ctas);
        for (int p = 0; p < net->n_buf && ok; ++p) {
            ok = cert::tc_make_map(&S.a_hi[p], net->buf[p], L.n_out, rows_max, L.ld_out, 128) &&
                 cert::tc_make_map(&S.a_lo[p], net->buf_lo[p], L.n_out, rows_max, L.ld_out, 128);
            if (ok && j > 0)
                ok = cert::tc_make_map(&S.o_hi[p], net->buf[p], L.ld_in, rows_max, L.ld_in, 32) &&
                     cert::tc_make_map(&S.o_lo[p], net->buf_lo[p], L.ld_in, rows_max, L.ld_in, 32);
        }
        if (!ok) break;
        {
            // y-major forms of what the start of a traversal at an FC layer right above needs
            be.assign(L.ld_out, 0.0f);
            for (int y = 0; y < L.h_out; ++y)
                for (int co = 0; co < L.c_out; ++co)
                    for (int x = 0; x < L.w_out; ++x) be[((size_t)y * L.c_out + co) * L.w_out + x] = descs[j].bias[co];
            if (!dev_alloc(net, (void **)&S.bias_out_y, be.size() * sizeof(float))) return CERT_ERR_OOM;
            if (cudaMemcpy(S.bias_out_y, be.data(), be.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                return CERT_ERR_CUDA;
            const LayerDev &La = net->layers[j + 1];
            if (La.kind == CERT_LAYER_FC) {
                const size_t rows_pad = round_up(La.n_out, kPad);
                hi.assign(rows_pad * La.ld_in, 0.0f);
                for (int i = 0; i < La.n_out; ++i)
                    for (int y = 0; y < L.h_out; ++y)
                        for (int co = 0; co < L.c_out; ++co)
                            for (int x = 0; x < L.w_out; ++x)
                                hi[(size_t)i * La.ld_in + ((size_t)y * L.c_out + co) * L.w_out + x] =
                                    descs[j + 1].weight[(size_t)i * La.n_in + ((size_t)co * L.h_out + y) * L.w_out + x];
                if (!dev_alloc(net, (void **)&S.W_above_y, hi.size() * sizeof(float))) return CERT_ERR_OOM;
                if (cudaMemcpy(S.W_above_y, hi.data(), hi.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                    return CERT_ERR_CUDA;
            }
        }
        S.usable = true;
        net->d_slots = std::max(net->d_slots, S.n_bands * S.plan.n_tiles);
        net->gat_floats = std::max(net->gat_floats, (size_t)net->max_batch * std::max(L.ld_in, L.ld_out));
        net->band[j] = S;
    }
    // Nets with residual connections: a waiting matrix must be in the layout of the step it joins, which holds
    // when every layer a connection ends on is itself banded (its matrix is then y-major when it is set aside).
    for (int k = 0; k < K && !net->skip_from.empty(); ++k) {
        if (net->skip_from[k] < 0) continue;
        const LayerDev &D = net->layers[k], &S = net->layers[net->skip_from[k]];
        if (!net->band[k].usable || S.kind != CERT_LAYER_CONV2D || S.c_out != D.c_out || S.h_out != D.h_out ||
            S.w_out != D.w_out)
            net->band_residual_ok = false;            // (the two maps must share one y-major order)
    }
    return CERT_OK;
}

// Counts launches; with profiling on, drops an event after each so that the
// time between consecutive events is that launch's device time.
struct Recorder {
    cert_net *net;
    cudaStream_t st;
    int launches = 0, marks = 0;
    Recorder(cert_net *n, cudaStream_t s) : net(n), st(s) {
        if (net->profiling && !net->prof_events.empty()) cudaEventRecord(net->prof_events[0], st);
    }
    void mark(int cls) {
        ++launches;
        if (!net->profiling) return;
        if (marks + 1 >= (int)net->prof_events.size()) return;
        net->prof_class[marks] = cls;
        ++marks;
        cudaEventRecord(net->prof_events[marks], st);
    }
};

#ifdef CERT_BOUNDS
// Checking build: the table of writable buffers (every allocation of the net plus the caller's arrays) goes to
// every translation unit's device copy before a call's first launch.
std::vector<void (*)(const cert::BoundsTable *)> &bounds_uploaders() {
    static std::vector<void (*)(const cert::BoundsTable *)> v;
    return v;
}

cert_status_t bounds_sync(cert_net *net, const void *const *extra, const size_t *extra_bytes, int n_extra) {
    static cert::BoundsTable t;
    t.n = 0;
    t.status = net->status_dev;
    for (const cert_net::Guarded &g : net->guards) {
        if (t.n >= cert::kBoundsMax) return CERT_ERR_UNSUPPORTED;
        t.lo[t.n] = (unsigned long long)(g.base + kGuardBytes);
        t.hi[t.n] = t.lo[t.n] + g.bytes;
        ++t.n;
    }
    for (int i = 0; i < n_extra; ++i) {
        if (t.n >= cert::kBoundsMax) return CERT_ERR_UNSUPPORTED;
        t.lo[t.n] = (unsigned long long)extra[i];
        t.hi[t.n] = t.lo[t.n] + extra_bytes[i];
        ++t.n;
    }
    cert::bounds_upload_all(&t);
    if (cudaGetLastError() != cudaSuccess) return CERT_ERR_CUDA;
    return CERT_OK;
}
#endif

// ---- the per-call schedule: one function per way a layer's traversal can run ----

// What the schedules of one layer's traversal share.  The traversal of layer k's expressions goes through
// layers k-1 .. j_end and is then simplified against the concrete bounds of what it has reached: the box
// (j_end = 0), or the outputs of layer j_end-1.
struct Traversal {
    cert_net *net;
    cudaStream_t st;
    Recorder *rec;
    int mode;                 // the contraction mode of this traversal (AUTO resolved)
    int *status;              // the status word its kernels report to: the net's, or the layer's word of a speculative run
    bool on_trial = false;    // a speculative fp16 run (a flagged range is made good by the re-run behind it)
    const int *run_if;        // not null: a re-run whose kernels do nothing unless that word is non-zero
    int batch, k, j_end, steps;
    long long rows;           // 2 * batch * n_k, ordered (box, side, neuron)
    const float *box_l, *box_u;
    float *lb_out, *ub_out;
    int paths;                // bits of cert_net_last_contraction_paths this traversal sets

    const LayerDev &layer(int j) const { return net->layers[j]; }
    const LayerDev &Lk() const { return net->layers[k]; }
    bool residual() const { return !net->skip_from.empty(); }
    // Relu transformer of layer k; with `slots` its bounds are first summed from n_slots partial sums per row.
    void relax(const float *slots, int n_slots, int slot_npos = 0) const {
        cert::launch_relax(Lk(), lb_out, ub_out, net->n_total, batch, net->codes, net->n_relu, slots, n_slots,
                           net->slot_stride, st, slot_npos, run_if);
        rec->mark(CERT_CLASS_RELAX);
    }
};

// The coefficient buffer a step writes to: the other one of two, or, in a net with residual connections, the one
// of three that neither holds the current matrix nor the matrix a connection has set aside (`kept`, -1: none).
int next_buffer(const Traversal &t, int cur, int kept) {
    if (!t.residual()) return cur ^ 1;
    int nxt = 0;
    while (nxt == cur || nxt == kept) ++nxt;
    return nxt;
}

// Coefficients that wait on a residual connection's source (layer `wait_for`): the matrix in buffer `kept`,
// untouched meanwhile, or the unit coefficient of layer k's own connection (`identity`), until the step whose
// result is over that source's outputs, where they join before the ReLU back-step.
struct Waiting {
    int wait_for = -1;
    bool identity = false;
    int kept = -1;
    bool kept_pair = false;
    void start(const Traversal &t) {
        wait_for = t.residual() ? t.net->skip_from[t.k] : -1;
        identity = wait_for >= 0;
    }
    // the expression is over layer j's affine neurons = W_j a_{j-1} + b_j + a_s: its matrix stays where it is
    // as the coefficients on a_s
    void set_aside(const Traversal &t, int j, int cur, bool pair) {
        if (!t.residual() || t.net->skip_from[j] < 0) return;
        wait_for = t.net->skip_from[j];
        identity = false;
        kept = cur;
        kept_pair = pair;
    }
    void joined() { wait_for = -1; identity = false; kept = -1; }
};

// The fields every tensor-core launch of a traversal fills the same way: problem and tile sizes, the slots
// the row constants travel in, the status word.  panel_rows = rows of a work tile's row panel.
cert::TcArgs tc_args(const Traversal &t, int K, int n_k, int ld_n, int bn, int n_tiles, int stages, int tmem_cols,
                     int panel_rows, int tiles_per_panel, int dcur, int dslots) {
    cert::TcArgs a;
    std::memset(&a, 0, sizeof(a));
    a.M = t.rows; a.K = K; a.n_k = n_k; a.ld_n = ld_n;
    a.bn = bn; a.n_tiles = n_tiles; a.stages = stages; a.tmem_cols = tmem_cols;
    a.total_tiles = (int)cert::ceil_div_ll(t.rows, panel_rows) * tiles_per_panel;
    a.d_in = t.net->dbuf[dcur]; a.n_slots_in = dslots; a.d_out = t.net->dbuf[dcur ^ 1];
    a.slot_stride = t.net->slot_stride;
    a.status = t.status;
    a.run_if = t.run_if;
    return a;
}

// The ReLU back-step through the neurons below layer j (relaxation of layer j-1) as a contraction's epilogue.
void tc_relu_epilogue(cert::TcArgs &a, const LayerDev &Lb, bool split_out) {
    a.has_relu = Lb.relu_after;
    a.split_out = split_out ? 1 : 0;
    a.lamL = Lb.lamL; a.lamU = Lb.lamU; a.nuU = Lb.nuU; a.bias_below = Lb.bias_n;
}

// No traversal at all: the interval step of W_k against the bounds of the layer below (IBP listing).
void run_interval_step(Traversal &t) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk(), &Lb = t.layer(t.k - 1);
    cert::launch_first_layer_bounds(Lk, Lb.actL, Lb.actU, Lb.ld_out, t.batch, t.lb_out, t.ub_out, net->n_total, t.st);
    t.rec->mark(CERT_CLASS_CONCRETIZE);
    if (t.residual() && net->skip_from[t.k] >= 0) {
        cert::launch_add_act_bounds(Lk, t.layer(net->skip_from[t.k]), t.batch, t.lb_out, t.ub_out, net->n_total, t.st);
        t.rec->mark(CERT_CLASS_CONCRETIZE);
    }
    if (Lk.relu_after || t.k + 1 < net->n_layers) t.relax(nullptr, 0);
}

// One-pass form of the fp16 split: the traversal's coefficients travel as pairs of 2^qa Q.  With a range proof the
// exponent is what the proved bound leaves of the fp16 range (up to kQaMax; the lo part of a coefficient is a normal
// fp16 number where |Q| 2^qa >= 2^-3); without one, a run on trial takes kQaTrial (a flagged
// range costs the re-run) and a forced run takes 0 (the whole fp16 range, as the two-pass form).
int fp16_scale_exponent(const Traversal &t) {
    const cert_net *net = t.net;
    if (!net->tc16_one_pass) return 0;
    const float b = t.k < (int)net->fp16_layer_bound.size() ? net->fp16_layer_bound[t.k] : INFINITY;
    if (std::isfinite(b) && b <= kFp16Safe) {
        int e = 0;
        std::frexp(kFp16Safe / std::max(b, 1e-30f), &e);          // ratio = m 2^e, m in [0.5, 1)
        return std::min(std::max(e - 1, 0), kQaMax);
    }
    return t.on_trial ? kQaTrial : 0;
}

// fp16 split, narrow FC nets: the whole traversal in one launch, the coefficient panel in shared memory.
void run_chain16(Traversal &t) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk();
    cert::ChainArgs a;
    std::memset(&a, 0, sizeof(a));
    a.M = t.rows; a.n_k = Lk.n_out; a.k = t.k; a.j_end = t.j_end;
    a.Wk = Lk.W; a.ldw_k = Lk.ld_in; a.bias_k = Lk.bias_n;
    a.box_l = t.box_l; a.box_u = t.box_u;
    a.d_out = net->dbuf[0]; a.slot_stride = net->slot_stride;
    a.status = t.status;
    a.stages = net->chain_stages; a.a_blocks = net->chain_a_blocks;
    a.b_chunk_bytes = net->chain_chunk; a.vec_ld = net->chain_vec_ld;
    const int qa = fp16_scale_exponent(t);
    a.one_pass = net->tc16_one_pass ? 1 : 0;
    a.q_scale = std::ldexp(1.0f, qa); a.q_unscale = std::ldexp(1.0f, -qa);
    const int pairs = (int)std::min<long long>(cert::ceil_div_ll(t.rows, 256), net->sm_count / 2);
    cert::launch_chain16(net->chain, a, pairs, net->chain_smem, t.st);
    t.rec->mark(CERT_CLASS_AFFINE);
    t.relax(net->dbuf[0], cert::kChainColGroups);
    t.paths |= 2 | 4 | 16 | 32;
}

// fp16 split, FC nets: the start, then one contraction per layer with the ReLU back-step fused, the last one
// concretising.  Residual connections as in run_dense: the waiting matrix keeps its buffer.
void run_tc16_steps(Traversal &t) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk();
    __half *qh[3], *ql[3];
    for (int p = 0; p < 3; ++p) {
        qh[p] = reinterpret_cast<__half *>(net->buf[p]);
        ql[p] = reinterpret_cast<__half *>(net->buf_lo[p]);
    }
    const bool one_pass = net->tc16_one_pass;
    const int qa = fp16_scale_exponent(t);
    const float q_scale = std::ldexp(1.0f, qa), q_unscale = std::ldexp(1.0f, -qa);
    int cur = 0, dcur = 0, dslots = 1;
    cert::launch_init_expr16(Lk, t.layer(t.k - 1), t.batch, qh[cur], ql[cur], net->dbuf[dcur], t.status,
                             one_pass ? q_scale : 1.0f, one_pass ? 1.0f : cert::kLoScale, t.st);
    t.rec->mark(CERT_CLASS_RELU_STEP);
    Waiting w;
    w.start(t);
    for (int j = t.k - 1; j >= t.j_end; --j) {
        const LayerDev &Lj = t.layer(j);
        const Tc16Layer &T = net->tc16[j];
        w.set_aside(t, j, cur, true);
        const int nxt = next_buffer(t, cur, w.kept);
        const bool join = j > t.j_end && w.wait_for == j - 1;
        // the tile plan: 256-column tiles unless the row panels are too few to give every CTA pair one; then as many
        // column tiles as keep the launch one wave of work tiles
        const cert::Tc16Plan *P = &T.plan;
        const cert::TcMap *b_hi = one_pass ? &T.s_hi : &T.b_hi, *b_lo = one_pass ? &T.s_lo : &T.b_lo;
        const long long panels = cert::ceil_div_ll(t.rows, 256);
        const int want = (int)std::min<long long>((net->sm_count / 2) / panels, kMaxFineTiles);
        if (one_pass && want > T.plan.n_tiles && !T.finer.empty()) {
            const int i = std::min(want - T.plan.n_tiles - 1, (int)T.finer.size() - 1);
            if (T.finer[i].ok) { P = &T.finer[i].plan; b_hi = &T.finer[i].hi; b_lo = &T.finer[i].lo; }
        }
        cert::TcArgs a = tc_args(t, Lj.n_out, Lk.n_out, Lj.ld_in, P->bn, P->n_tiles, P->stages, P->tmem_cols, 256,
                                 P->n_tiles, dcur, dslots);
        a.q_scale = q_scale; a.q_unscale = q_unscale; a.acc_scale = q_unscale * T.w_unscale;
        a.n_narrow = P->n_narrow;
        const int pairs = std::min(a.total_tiles, net->sm_count / 2);
        if (j > t.j_end) {
            tc_relu_epilogue(a, t.layer(j - 1), true);
            if (join && w.kept >= 0) {
                a.add_hi = reinterpret_cast<const float *>(qh[w.kept]);
                a.add_lo = reinterpret_cast<const float *>(ql[w.kept]);
            }
            a.add_identity = (join && w.identity) ? 1 : 0;
            cert::launch_gemm_tc16(cert::TC_EPI_RELU, one_pass, pairs, T.a_hi[cur], T.a_lo[cur], *b_hi, *b_lo, T.o_hi[nxt],
                                   T.o_lo[nxt], a, P->smem_bytes, t.st);
            if (join) w.joined();
        } else {
            a.l0 = t.box_l; a.u0 = t.box_u;
            cert::launch_gemm_tc16(cert::TC_EPI_CONCRETIZE, one_pass, pairs, T.a_hi[cur], T.a_lo[cur], *b_hi, *b_lo,
                                   T.a_hi[cur], T.a_lo[cur], a, P->smem_bytes, t.st);
        }
        t.rec->mark(CERT_CLASS_AFFINE);
        cur = nxt;
        dcur ^= 1;
        dslots = 2 * P->n_tiles;
    }
    t.relax(net->dbuf[dcur], dslots);
    t.paths |= 2 | 4 | 16;
}

// A conv layer over conv layers, rows as receptive-field patches, every step as a contraction with the conv
// layer's window-to-window matrix on the tensor cores.
void run_patches_tc(Traversal &t, const cert::PatchLevel *lv) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk();
    const std::vector<TcPatchStep> &SS = net->tcp[t.k];
    const int ctas = net->tc_ctas;
    int cur = 0, dcur = 0, dslots = 1;
    cert::launch_patch_start(Lk, t.layer(t.k - 1), SS[0].Kp, t.batch, net->buf[cur], net->buf_lo[cur], net->dbuf[dcur],
                             t.st);
    t.rec->mark(CERT_CLASS_RELU_STEP);
    for (int j = t.k - 1, m = 0; j >= t.j_end; --j, ++m) {
        const LayerDev &Lj = t.layer(j);
        const TcPatchStep &S = SS[m];
        const float *src[3] = {nullptr, nullptr, nullptr};
        const float fill[3] = {1.0f, 1.0f, 0.0f};
        int n_arr = 3;
        if (j > t.j_end) {
            const LayerDev &Lb = t.layer(j - 1);
            if (Lb.relu_after) { src[0] = Lb.lamL; src[1] = Lb.lamU; src[2] = Lb.nuU; }
        } else {
            src[0] = t.box_l; src[1] = t.box_u;
            n_arr = 2;
        }
        cert::launch_patch_gather(Lk, Lj, lv[m + 1], S.ldN, t.batch, n_arr, src, fill, net->gat, t.st);
        t.rec->mark(CERT_CLASS_CONV);
        // rows are ordered (box, position, side, channel): with "box" = (box, position) and c_out neurons
        // per box this is the usual row order, and the gathered vectors are per such box
        cert::TcArgs a = tc_args(t, S.Kp, Lk.c_out, S.ldN, S.plan.bn, S.plan.n_tiles, S.plan.stages, S.plan.tmem_cols,
                                 128 * ctas, S.plan.n_tiles, dcur, dslots);
        const int groups = std::min(a.total_tiles, net->sm_count / ctas);
        if (j > t.j_end) {
            a.has_relu = 1;          // the gathered slopes also blank the window outside the map
            a.split_out = 1;
            a.lamL = net->gat[0]; a.lamU = net->gat[1]; a.nuU = net->gat[2]; a.bias_below = S.bias_e;
            cert::launch_gemm_tc(cert::TC_EPI_RELU, ctas, groups, S.a_hi[cur], S.a_lo[cur], S.b_hi, S.b_lo,
                                 S.o_hi[cur ^ 1], S.o_lo[cur ^ 1], a, S.plan.smem_bytes, t.st);
        } else {
            a.l0 = net->gat[0]; a.u0 = net->gat[1];
            cert::launch_gemm_tc(cert::TC_EPI_CONCRETIZE, ctas, groups, S.a_hi[cur], S.a_lo[cur], S.b_hi, S.b_lo,
                                 S.a_hi[cur], S.a_lo[cur], a, S.plan.smem_bytes, t.st);
        }
        t.rec->mark(CERT_CLASS_CONV);
        cur ^= 1;
        dcur ^= 1;
        dslots = S.plan.n_tiles;
    }
    t.relax(net->dbuf[dcur], dslots, Lk.h_out * Lk.w_out);
    t.paths |= 8 | 2 | (ctas == 2 ? 4 : 0);
}

// The same traversal with the patch steps on the FMA units (one warp per row).
void run_patches_fma(Traversal &t, const cert::PatchLevel *lv) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk();
    int cur = 0;
    const int dcur = 0;
    cert::launch_patch_start(Lk, t.layer(t.k - 1), lv[0].pitch, t.batch, net->buf[cur], nullptr, net->dbuf[dcur], t.st);
    t.rec->mark(CERT_CLASS_RELU_STEP);
    for (int j = t.k - 1, m = 0; j >= t.j_end; --j, ++m) {
        cert::ConvtEpilogue ep;
        std::memset(&ep, 0, sizeof(ep));
        ep.n_k = Lk.n_out;
        ep.d_in = net->dbuf[dcur]; ep.n_slots_in = 1; ep.slot_stride = net->slot_stride;
        ep.d_out = net->dbuf[dcur];
        if (j > t.j_end) {
            const LayerDev &Lb = t.layer(j - 1);
            ep.mode = cert::CONVT_EPI_RELU;
            ep.has_relu = Lb.relu_after;
            ep.lamL = Lb.lamL; ep.lamU = Lb.lamU; ep.nuU = Lb.nuU; ep.bias_below = Lb.bias_n;
            ep.P = net->buf[cur ^ 1];
        } else {
            ep.mode = cert::CONVT_EPI_CONCRETIZE;
            ep.l0 = t.box_l; ep.u0 = t.box_u;
            ep.lb_out = t.lb_out; ep.ub_out = t.ub_out; ep.n_total = net->n_total; ep.out_off = Lk.out_off;
        }
        cert::launch_patch_step(Lk, t.layer(j), lv[m], lv[m + 1], net->buf[cur], t.rows, net->sm_count, ep, t.st);
        t.rec->mark(CERT_CLASS_CONV);
        cur ^= 1;
    }
    if (Lk.relu_after || t.k + 1 < net->n_layers) t.relax(nullptr, 0);
    t.paths |= 8;
}

// Everything else: dense coefficient matrices, one launch per back-step (3xTF32 contraction, banded conv form,
// FMA conv kernel, or the FMA chain of contraction + ReLU step), residual connections included.
void run_dense(Traversal &t) {
    cert_net *net = t.net;
    const LayerDev &Lk = t.Lk();
    const int K = net->n_layers, k = t.k, j_end = t.j_end, n_total = net->n_total;
    const bool residual = t.residual();
    cudaStream_t st = t.st;
    Recorder &rec = *t.rec;
    int cur = 0;      // coefficient buffer that holds the current expression
    int dcur = 0;     // constant buffer, and how many of its slots are live
    int dslots = 1;
    bool bounds_in_slots = false;
    // Does the back-step through layer j run on the tensor cores?  Its input must then be a TF32 pair.
    auto on_tc = [&](int j) { return t.mode != CERT_CONTRACTION_FFMA && net->tc_ok && net->tc[j].usable; };
    // ... or, for a conv layer on dense maps, in the banded tensor-core form?  Its input is a TF32 pair too.
    auto on_band = [&](int j) {
        return t.mode != CERT_CONTRACTION_FFMA && net->tc_ok && net->band[j].usable &&
               (!residual || (net->band_residual_ok && t.steps == k));      // (residual nets: full traversals)
    };
    auto wants_pair = [&](int j) { return on_tc(j) || on_band(j); };

    // expression over the outputs of layer k-1, pushed through its ReLU
    bool y_major = false;     // the coefficient maps are held [y][channel][x] (banded conv steps)
    if (Lk.kind == CERT_LAYER_FC && on_band(k - 1) && net->band[k - 1].W_above_y) {
        // an FC layer right above a banded conv layer: the same start with the columns of W_k, the relaxation
        // and the bias below in y-major order writes the first matrix in the layout the banded steps read
        const LayerDev &Lb = t.layer(k - 1);
        const BandStep &S = net->band[k - 1];
        const float *src[3] = {nullptr, nullptr, nullptr};
        const float fill[3] = {1.0f, 1.0f, 0.0f};
        if (Lb.relu_after) { src[0] = Lb.lamL; src[1] = Lb.lamU; src[2] = Lb.nuU; }
        cert::launch_to_ymajor_vectors(Lb.c_out, Lb.h_out, Lb.w_out, Lb.ld_out, t.batch, 3, src, fill, net->gat, st);
        rec.mark(CERT_CLASS_RELU_STEP);
        LayerDev Lk_y = Lk, Lb_y = Lb;
        Lk_y.W = S.W_above_y;
        Lb_y.lamL = net->gat[0]; Lb_y.lamU = net->gat[1]; Lb_y.nuU = net->gat[2];
        Lb_y.bias_n = S.bias_out_y;
        Lb_y.relu_after = 1;
        cert::launch_init_expr(Lk_y, Lb_y, t.batch, net->buf[cur], net->buf_lo[cur], net->dbuf[dcur], st);
        y_major = true;
    } else {
        // a conv layer right above a banded conv layer places its window coefficients at their y-major columns
        y_major = Lk.kind == CERT_LAYER_CONV2D && on_band(k - 1);
        cert::launch_init_expr(Lk, t.layer(k - 1), t.batch, net->buf[cur],
                               wants_pair(k - 1) ? net->buf_lo[cur] : nullptr, net->dbuf[dcur], st, y_major, t.run_if);
    }
    rec.mark(CERT_CLASS_RELU_STEP);
    Waiting w;
    w.start(t);
    for (int j = k - 1; j >= j_end; --j) {
        const LayerDev &Lj = t.layer(j);
        w.set_aside(t, j, cur, wants_pair(j));
        int nxt = next_buffer(t, cur, w.kept);
        // The last step of a traversal that stops on the very neurons a connection waits for: the
        // coefficients join before the simplification, so the step stores its result and the unfused
        // concretisation follows.
        const bool join_end = residual && j == j_end && j_end > 0 && w.wait_for == j_end - 1;
        const bool join = (j > j_end && w.wait_for == j - 1) || join_end;
        const bool store_step = j > j_end || join_end;
        const float *add_hi = (join && w.kept >= 0) ? net->buf[w.kept] : nullptr;
        const float *add_lo = (join && w.kept >= 0 && w.kept_pair) ? net->buf_lo[w.kept] : nullptr;
        const int add_identity = (join && w.identity) ? 1 : 0;
        if (Lj.kind == CERT_LAYER_CONV2D && on_band(j)) {
            // dense coefficient maps through conv layer j on the tensor cores, band by band
            const BandStep &S = net->band[j];
            const int ctas = net->tc_ctas;
            if (!y_major) {
                cert::launch_to_ymajor_pair(net->buf[cur], net->buf_lo[cur], net->buf[nxt], net->buf_lo[nxt], t.rows,
                                            Lj.c_out, Lj.h_out, Lj.w_out, Lj.ld_out, st);
                rec.mark(CERT_CLASS_CONV);
                if (w.kept == cur) w.kept = nxt;      // a matrix set aside at this very layer: its y-major copy waits
                cur = nxt;
                nxt = next_buffer(t, cur, w.kept);
                y_major = true;
            }
            const float *src[3] = {nullptr, nullptr, nullptr};
            const float fill[3] = {1.0f, 1.0f, 0.0f};
            int n_arr = 3;
            if (j > j_end) {
                const LayerDev &Lb = t.layer(j - 1);
                if (Lb.relu_after) { src[0] = Lb.lamL; src[1] = Lb.lamU; src[2] = Lb.nuU; }
            } else {
                src[0] = t.box_l; src[1] = t.box_u;
                n_arr = 2;
            }
            cert::launch_to_ymajor_vectors(Lj.c_in, Lj.h_in, Lj.w_in, Lj.ld_in, t.batch, n_arr, src, fill, net->gat, st);
            rec.mark(CERT_CLASS_CONV);
            cert::TcArgs a = tc_args(t, S.K, Lk.n_out, Lj.ld_in, S.plan.bn, S.plan.n_tiles, S.plan.stages,
                                     S.plan.tmem_cols, 128 * ctas, S.n_bands * S.plan.n_tiles, dcur, dslots);
            a.n_bands = S.n_bands; a.band_rin = S.rin; a.band_o_shift = S.o_shift; a.band_h_in = Lj.h_out;
            a.band_row_in = Lj.c_out * Lj.w_out;
            a.band_s = Lj.stride; a.band_y_shift = S.y_shift; a.band_row_out = Lj.c_in * Lj.w_in;
            const int groups = std::min(a.total_tiles, net->sm_count / ctas);
            if (j > j_end) {
                a.has_relu = 1;
                a.split_out = 1;          // a banded step follows
                a.lamL = net->gat[0]; a.lamU = net->gat[1]; a.nuU = net->gat[2]; a.bias_below = S.bias_y;
                if (join && w.kept >= 0) { a.add_hi = net->buf[w.kept]; a.add_lo = net->buf_lo[w.kept]; }
                a.add_identity = add_identity;
                a.band_c_out = Lj.c_in; a.band_h_out = Lj.h_in; a.band_w_out = Lj.w_in;
                cert::launch_gemm_tc(cert::TC_EPI_RELU_BAND, ctas, groups, S.a_hi[cur], S.a_lo[cur], S.b_hi, S.b_lo,
                                     S.o_hi[nxt], S.o_lo[nxt], a, S.plan.smem_bytes, st);
                if (join) w.joined();
            } else {
                a.l0 = net->gat[0]; a.u0 = net->gat[1];
                cert::launch_gemm_tc(cert::TC_EPI_CONCRETIZE_BAND, ctas, groups, S.a_hi[cur], S.a_lo[cur], S.b_hi,
                                     S.b_lo, S.a_hi[cur], S.a_lo[cur], a, S.plan.smem_bytes, st);
                bounds_in_slots = true;
            }
            rec.mark(CERT_CLASS_CONV);
            t.paths |= 2 | (ctas == 2 ? 4 : 0) | 64;
            cur = nxt;
            dcur ^= 1;
            dslots = S.n_bands * S.plan.n_tiles;
            continue;
        }
        float *Q = net->buf[cur], *P = net->buf[nxt];
        float *P_lo = (j > j_end && wants_pair(j - 1)) ? net->buf_lo[nxt] : nullptr;
        if (on_tc(j)) {
            const TcLayer &T = net->tc[j];
            const int ctas = net->tc_ctas;
            cert::TcArgs a = tc_args(t, Lj.n_out, Lk.n_out, Lj.ld_in, T.plan.bn, T.plan.n_tiles, T.plan.stages,
                                     T.plan.tmem_cols, 128 * ctas, T.plan.n_tiles, dcur, dslots);
            const int groups = std::min(a.total_tiles, net->sm_count / ctas);
            if (store_step) {
                tc_relu_epilogue(a, t.layer(j - 1), P_lo != nullptr);
                if (join_end) { a.has_relu = 0; a.bias_below = net->zeros; }
                a.add_hi = add_hi; a.add_lo = add_lo; a.add_identity = add_identity;
                cert::launch_gemm_tc(cert::TC_EPI_RELU, ctas, groups, T.a_hi[cur], T.a_lo[cur], T.b_hi, T.b_lo,
                                     T.o_hi[nxt], T.o_lo[nxt], a, T.plan.smem_bytes, st);
            } else {
                a.l0 = t.box_l; a.u0 = t.box_u;
                cert::launch_gemm_tc(cert::TC_EPI_CONCRETIZE, ctas, groups, T.a_hi[cur], T.a_lo[cur], T.b_hi, T.b_lo,
                                     T.a_hi[cur], T.a_lo[cur], a, T.plan.smem_bytes, st);
                bounds_in_slots = true;
            }
            rec.mark(CERT_CLASS_AFFINE);
            t.paths |= 2 | (ctas == 2 ? 4 : 0);
            if (join) w.joined();
            cur = nxt;
            dcur ^= 1;
            dslots = T.plan.n_tiles;
            if (join_end) {
                cert::launch_concretize(P, net->dbuf[dcur], dslots, net->slot_stride, t.box_l, t.box_u, Lj.n_in,
                                        Lj.ld_in, t.batch, Lk.n_out, t.lb_out, t.ub_out, n_total, Lk.out_off, st);
                rec.mark(CERT_CLASS_CONCRETIZE);
            }
            continue;
        }
        if (Lj.kind == CERT_LAYER_CONV2D) {
            // conv back-step with what follows it fused: the ReLU back-step below, or the concretisation
            cert::ConvtEpilogue ep;
            std::memset(&ep, 0, sizeof(ep));
            ep.n_k = Lk.n_out;
            ep.d_in = net->dbuf[dcur]; ep.n_slots_in = dslots; ep.slot_stride = net->slot_stride;
            ep.d_out = net->dbuf[dcur];
            if (store_step) {
                const LayerDev &Lb = t.layer(j - 1);
                ep.mode = cert::CONVT_EPI_RELU;
                ep.has_relu = join_end ? 0 : Lb.relu_after;
                ep.lamL = Lb.lamL; ep.lamU = Lb.lamU; ep.nuU = Lb.nuU;
                ep.bias_below = join_end ? net->zeros : Lb.bias_n;
                ep.P = P; ep.P_lo = P_lo;
                ep.add_hi = add_hi; ep.add_lo = add_lo; ep.add_identity = add_identity;
            } else {
                ep.mode = cert::CONVT_EPI_CONCRETIZE;
                ep.l0 = t.box_l; ep.u0 = t.box_u;
                ep.lb_out = t.lb_out; ep.ub_out = t.ub_out; ep.n_total = n_total; ep.out_off = Lk.out_off;
            }
            cert::launch_convt_ffma(Lj, Q, t.rows, net->sm_count, ep, st);
            rec.mark(CERT_CLASS_CONV);
            if (join) w.joined();
            cur = nxt;
            dslots = 1;
            if (join_end) {
                cert::launch_concretize(P, net->dbuf[dcur], dslots, net->slot_stride, t.box_l, t.box_u, Lj.n_in,
                                        Lj.ld_in, t.batch, Lk.n_out, t.lb_out, t.ub_out, n_total, Lk.out_off, st);
                rec.mark(CERT_CLASS_CONCRETIZE);
            }
            continue;
        }
        // FC layer on the FMA units: contraction, then the ReLU back-step or the concretisation as kernels of their own
        cert::launch_gemm_ffma(Q, Lj.ld_out, Lj.W, Lj.ld_in, P, Lj.ld_in, t.rows, Lj.n_in, Lj.n_out, st);
        rec.mark(CERT_CLASS_AFFINE);
        t.paths |= 1;
        cur = nxt;
        if (join) {
            cert::launch_add_skip(P, add_hi, add_lo, add_identity, t.rows, Lj.n_in, Lj.ld_in, Lk.n_out, st);
            rec.mark(CERT_CLASS_RELU_STEP);
            w.joined();
        }
        if (j > j_end) {
            cert::launch_relu_step(t.layer(j - 1), t.batch, Lk.n_out, P, P_lo, net->dbuf[dcur], dslots,
                                   net->slot_stride, st);
            dslots = 1;
            rec.mark(CERT_CLASS_RELU_STEP);
        } else {
            cert::launch_concretize(P, net->dbuf[dcur], dslots, net->slot_stride, t.box_l, t.box_u, Lj.n_in, Lj.ld_in,
                                    t.batch, Lk.n_out, t.lb_out, t.ub_out, n_total, Lk.out_off, st);
            rec.mark(CERT_CLASS_CONCRETIZE);
        }
    }
    if (residual && w.wait_for >= 0) {
        // the traversal stopped above the connection's source: the waiting neurons are simplified against
        // their own concrete bounds
        const float *S_hi = w.kept >= 0 ? net->buf[w.kept] : nullptr;
        const float *S_lo = (w.kept >= 0 && w.kept_pair) ? net->buf_lo[w.kept] : nullptr;
        float *slot = nullptr;
        if (bounds_in_slots) {
            slot = net->dbuf[dcur] + (size_t)dslots * net->slot_stride;
            ++dslots;
        }
        cert::launch_skip_concretize(S_hi, S_lo, w.identity ? 1 : 0, t.layer(w.wait_for), t.rows, Lk, slot, t.lb_out,
                                     t.ub_out, n_total, st);
        rec.mark(CERT_CLASS_CONCRETIZE);
    }
    if (Lk.relu_after || bounds_in_slots || k + 1 < K) t.relax(bounds_in_slots ? net->dbuf[dcur] : nullptr, dslots);
}

// The contraction mode the traversal of layer k runs in.  AUTO: the fp16 split where the net's weights prove that
// no coefficient of that traversal can leave the fp16 range (cert_net::fp16_layer_bound), else the TF32 split;
// `forced` >= 0 overrides the net's setting.
int layer_mode(const cert_net *net, int forced, int k) {
    const int mode = forced >= 0 ? forced : net->contraction;
    if (mode == CERT_CONTRACTION_AUTO && net->tc16_ok && k < (int)net->fp16_layer_bound.size() &&
        net->fp16_layer_bound[k] <= kFp16Safe)
        return CERT_CONTRACTION_TC3XFP16;
    return mode;
}

// flow(forward) over the layers: the bounds of the first layer against the box, then for every affine layer its
// traversal in whichever schedule takes it, then the Relu transformer.
cert_status_t backsub_impl(cert_net *net, const float *centers, float eps, int batch, const int *backsteps,
                           float *lb_out, float *ub_out, cudaStream_t st, int forced_mode) {
    if (!net || !centers || !lb_out || !ub_out) return CERT_ERR_INVALID_ARG;
    if (batch < 1 || !(eps >= 0.0f) || std::isinf(eps)) return CERT_ERR_INVALID_ARG;
    if (batch > net->max_batch) return CERT_ERR_BATCH_TOO_LARGE;
    const int K = net->n_layers;
    const bool residual = !net->skip_from.empty();
    if (residual && backsteps && (forced_mode >= 0 ? forced_mode : net->contraction) == CERT_CONTRACTION_TC3XFP16)
        for (int k = 1; k < K; ++k)
            if (backsteps[k] >= 0 && backsteps[k] < k) return CERT_ERR_UNSUPPORTED;   // fp16 split: full traversals only
#ifdef CERT_BOUNDS
    {
        const void *extra[2] = {lb_out, ub_out};
        const size_t bytes[2] = {(size_t)batch * net->n_total * sizeof(float), (size_t)batch * net->n_total * sizeof(float)};
        const cert_status_t bs = bounds_sync(net, extra, bytes, 2);
        if (bs != CERT_OK) return bs;
    }
#endif
    Recorder rec(net, st);
    int paths = 0;

    cert::launch_box(centers, eps, net->clip_lo, net->clip_hi, batch, net->n0, net->ld0, net->l0, net->u0, st);
    rec.mark(CERT_CLASS_INPUT);
    cert::launch_first_layer_bounds(net->layers[0], net->l0, net->u0, net->ld0, batch, lb_out, ub_out, net->n_total, st);
    rec.mark(CERT_CLASS_INPUT);
    if (net->layers[0].relu_after || K > 1) {
        cert::launch_relax(net->layers[0], lb_out, ub_out, net->n_total, batch, net->codes, net->n_relu, nullptr, 0, 0,
                           st);
        rec.mark(CERT_CLASS_RELAX);
    }
    bool spec_cleared = false;
    for (int k = 1; k < K; ++k) {
        const int mode = layer_mode(net, forced_mode, k);
        Traversal t;
        t.net = net; t.st = st; t.rec = &rec; t.mode = mode; t.batch = batch; t.k = k;
        t.status = net->status_dev; t.run_if = nullptr;
        t.steps = (backsteps && backsteps[k] >= 0) ? std::min(backsteps[k], k) : k;
        t.j_end = k - t.steps;
        t.rows = 2LL * batch * net->layers[k].n_out;
        t.box_l = t.j_end == 0 ? net->l0 : net->layers[t.j_end - 1].actL;
        t.box_u = t.j_end == 0 ? net->u0 : net->layers[t.j_end - 1].actU;
        t.lb_out = lb_out; t.ub_out = ub_out;
        t.paths = 0;
        cert::PatchLevel lv[kMaxPatchLevels];
        // AUTO on a layer whose range proof failed: the fp16 split first, on its own status word, then the
        // predicated TF32 traversal (cert_net::speculate)
        // (nets with residual connections: the fp16 schedule covers full traversals only)
        const bool speculative = forced_mode < 0 && net->contraction == CERT_CONTRACTION_AUTO && net->speculate &&
                                 mode == CERT_CONTRACTION_AUTO && t.steps > 0 && (!residual || t.steps == k);
        if (speculative) {
            if (!spec_cleared) {
                if (cudaMemsetAsync(net->spec_dev, 0, (size_t)K * sizeof(int), st) != cudaSuccess) {
                    cudaGetLastError();
                    return CERT_ERR_CUDA;
                }
                spec_cleared = true;
            }
            t.mode = CERT_CONTRACTION_TC3XFP16;
            t.status = net->spec_dev + k;
            t.on_trial = true;
            if (net->chain_ok) run_chain16(t);
            else run_tc16_steps(t);
            t.on_trial = false;
            t.mode = CERT_CONTRACTION_TC3XTF32;
            t.status = net->status_dev;
            t.run_if = net->spec_dev + k;
            run_dense(t);
            paths |= t.paths | 128;
            continue;
        }
        if (t.steps == 0) {
            run_interval_step(t);
        } else if (mode == CERT_CONTRACTION_TC3XFP16 && net->chain_ok) {
            run_chain16(t);
        } else if (mode == CERT_CONTRACTION_TC3XFP16 && net->tc16_ok) {
            run_tc16_steps(t);
        } else if (net->conv_patches && cert::conv_patch_plan(net->layers.data(), k, t.j_end, lv, kMaxPatchLevels)) {
            if (mode != CERT_CONTRACTION_FFMA && (int)net->tcp[k].size() >= t.steps) run_patches_tc(t, lv);
            else run_patches_fma(t, lv);
        } else {
            run_dense(t);
        }
        paths |= t.paths;
    }
    net->last_batch = batch;
    net->last_launches = rec.launches;
    net->last_paths = paths;
    net->prof_marks = rec.marks;
    if (cudaPeekAtLastError() != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}

}  // namespace

extern "C" {

const char *cert_status_string(cert_status_t s) {
    switch (s) {
        case CERT_OK: return "ok";
        case CERT_ERR_INVALID_ARG: return "invalid argument";
        case CERT_ERR_UNSUPPORTED: return "unsupported";
        case CERT_ERR_OOM: return "out of memory";
        case CERT_ERR_BATCH_TOO_LARGE: return "batch larger than max_batch";
        case CERT_ERR_CUDA: return "CUDA error";
        case CERT_ERR_TIMEOUT: return "device-side wait timed out";
        case CERT_ERR_RANGE: return "coefficient outside the fp16 range of the TC3XFP16 contraction";
        case CERT_ERR_BOUNDS: return "a checked store fell outside every buffer (checking build)";
    }
    return "unknown";
}

static cert_status_t create_impl(const cert_layer_desc_t *layers, int n_layers, const int *skip_from, int max_batch,
                                 float clip_lo, float clip_hi, cert_net_t **out, cert_net **partial) {
    cert_status_t v = validate(layers, n_layers, max_batch, clip_lo, clip_hi);
    if (v != CERT_OK) return v;
    bool any_skip = false;
    if (skip_from) {
        // a connection spans at least one layer, joins equal widths, and connections follow one another
        // (none starts inside another's span)
        int last_end = 0;
        for (int k = 0; k < n_layers; ++k) {
            const int s = skip_from[k];
            if (s < 0) continue;
            if (s > k - 2 || s < last_end) return CERT_ERR_INVALID_ARG;
            const int n_s = layers[s].kind == CERT_LAYER_FC ? layers[s].out_features : desc_conv_out(layers[s]);
            const int n_k = layers[k].kind == CERT_LAYER_FC ? layers[k].out_features : desc_conv_out(layers[k]);
            if (n_s != n_k) return CERT_ERR_INVALID_ARG;
            last_end = k;
            any_skip = true;
        }
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CERT_ERR_CUDA; }

    cert_net *net = new (std::nothrow) cert_net;
    if (!net) return CERT_ERR_OOM;
    *partial = net;                     // the caller frees it if anything below throws
    net->device = dev;
    {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) == cudaSuccess) net->sm_count = prop.multiProcessorCount;
        else cudaGetLastError();
    }
    net->n_layers = n_layers;
    if (any_skip) {
        net->skip_from.assign(skip_from, skip_from + n_layers);
        net->n_buf = 3;
        net->conv_patches = false;
    }
    net->max_batch = max_batch;
    net->clip_lo = clip_lo;
    net->clip_hi = clip_hi;
    net->layers.resize(n_layers);

    cert_status_t fail = CERT_OK;
    int out_off = 0, relu_off = 0;
    std::vector<float> host;
    for (int k = 0; k < n_layers && fail == CERT_OK; ++k) {
        const cert_layer_desc_t &D = layers[k];
        LayerDev &L = net->layers[k];
        std::memset(&L, 0, sizeof(L));
        L.kind = D.kind;
        L.relu_after = D.relu_after;
        if (D.kind == CERT_LAYER_FC) {
            L.n_in = D.in_features;
            L.n_out = D.out_features;
        } else {
            L.c_in = D.c_in; L.h_in = D.h_in; L.w_in = D.w_in; L.c_out = D.c_out;
            L.kh = D.kh; L.kw = D.kw; L.stride = D.stride; L.pad = D.pad;
            L.h_out = (D.h_in + 2 * D.pad - D.kh) / D.stride + 1;
            L.w_out = (D.w_in + 2 * D.pad - D.kw) / D.stride + 1;
            L.n_in = D.c_in * D.h_in * D.w_in;
            L.n_out = D.c_out * L.h_out * L.w_out;
        }
        L.ld_in = round_up(L.n_in, kPad);
        L.ld_out = round_up(L.n_out, kPad);
        L.out_off = out_off;
        out_off += L.n_out;
        L.relu_off = relu_off;
        if (L.relu_after) relu_off += L.n_out;

        // per-neuron bias, zero padded
        host.assign(L.ld_out, 0.0f);
        if (D.kind == CERT_LAYER_FC) {
            for (int i = 0; i < L.n_out; ++i) host[i] = D.bias[i];
        } else {
            int hw = L.h_out * L.w_out;
            for (int i = 0; i < L.n_out; ++i) host[i] = D.bias[i / hw];
        }
        if (!dev_alloc(net, (void **)&L.bias_n, host.size() * sizeof(float))) { fail = CERT_ERR_OOM; break; }
        if (cudaMemcpy(L.bias_n, host.data(), host.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
            fail = CERT_ERR_CUDA; break;
        }

        if (D.kind == CERT_LAYER_FC) {
            size_t rows_pad = round_up(L.n_out, kPad);
            host.assign(rows_pad * L.ld_in, 0.0f);
            for (int i = 0; i < L.n_out; ++i)
                std::memcpy(&host[(size_t)i * L.ld_in], D.weight + (size_t)i * L.n_in, sizeof(float) * L.n_in);
            if (!dev_alloc(net, (void **)&L.W, host.size() * sizeof(float))) { fail = CERT_ERR_OOM; break; }
            if (cudaMemcpy(L.W, host.data(), host.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
                fail = CERT_ERR_CUDA; break;
            }
        } else {
            size_t nw = (size_t)L.c_out * L.c_in * L.kh * L.kw;
            if (!dev_alloc(net, (void **)&L.W, nw * sizeof(float))) { fail = CERT_ERR_OOM; break; }
            if (cudaMemcpy(L.W, D.weight, nw * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
                fail = CERT_ERR_CUDA; break;
            }
            host.assign(nw, 0.0f);
            for (int co = 0; co < L.c_out; ++co)
                for (int ci = 0; ci < L.c_in; ++ci)
                    for (int ky = 0; ky < L.kh; ++ky)
                        for (int kx = 0; kx < L.kw; ++kx)
                            host[(((size_t)co * L.kh + ky) * L.kw + kx) * L.c_in + ci] =
                                D.weight[(((size_t)co * L.c_in + ci) * L.kh + ky) * L.kw + kx];
            if (!dev_alloc(net, (void **)&L.Wct, nw * sizeof(float))) { fail = CERT_ERR_OOM; break; }
            if (cudaMemcpy(L.Wct, host.data(), nw * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
                fail = CERT_ERR_CUDA; break;
            }
            if (!cert::convt_supported(L)) { fail = CERT_ERR_UNSUPPORTED; break; }
        }
        if (L.relu_after) {
            size_t n = (size_t)max_batch * L.ld_out;
            if (!dev_alloc_zero(net, &L.lamL, n) || !dev_alloc_zero(net, &L.lamU, n) ||
                !dev_alloc_zero(net, &L.nuU, n)) { fail = CERT_ERR_OOM; break; }
        }
        if (k + 1 < n_layers) {
            size_t n = (size_t)max_batch * L.ld_out;
            if (!dev_alloc_zero(net, &L.actL, n) || !dev_alloc_zero(net, &L.actU, n)) { fail = CERT_ERR_OOM; break; }
        }
    }
    if (fail == CERT_OK) {
        net->n0 = net->layers[0].n_in;
        net->ld0 = net->layers[0].ld_in;
        net->n_total = out_off;
        net->n_relu = relu_off;
        // workspace: the largest coefficient matrix any traversal holds
        size_t max_elems = 1, max_rows = 1;
        for (int k = 1; k < n_layers; ++k) {
            size_t rows = 2ull * max_batch * net->layers[k].n_out;
            int ld_max = 0;
            for (int j = 0; j < k; ++j) {
                ld_max = std::max(ld_max, net->layers[j].ld_out);
                ld_max = std::max(ld_max, net->layers[j].ld_in);
            }
            max_elems = std::max(max_elems, rows * (size_t)ld_max);
            max_rows = std::max(max_rows, rows);
        }
        size_t b = (size_t)max_batch;
        bool ok = dev_alloc_zero(net, &net->l0, b * net->ld0) && dev_alloc_zero(net, &net->u0, b * net->ld0) &&
                  dev_alloc_zero(net, &net->buf[0], max_elems) && dev_alloc_zero(net, &net->buf[1], max_elems) &&
                  (net->n_buf < 3 || dev_alloc_zero(net, &net->buf[2], max_elems)) &&
                  dev_alloc_zero(net, &net->codes, b * std::max(1, net->n_relu)) &&
                  dev_alloc_zero(net, &net->status_dev, 1) &&
                  dev_alloc_zero(net, &net->centers_dev, b * net->n0) &&
                  dev_alloc_zero(net, &net->lb_dev, b * net->n_total) &&
                  dev_alloc_zero(net, &net->ub_dev, b * net->n_total);
        if (!ok) fail = CERT_ERR_OOM;
        net->slot_stride = (long long)max_rows;
        if (ok) fail = setup_tensor_core_path(net, layers, max_elems);
        if (ok && fail == CERT_OK) fail = prove_fp16_range(net);
        if (ok && fail == CERT_OK) fail = setup_patch_tc(net, layers);
        if (ok && fail == CERT_OK) fail = setup_band_tc(net, layers);
        if (ok && fail == CERT_OK && net->gat_floats)
            for (int i = 0; i < 3 && fail == CERT_OK; ++i)
                if (!dev_alloc_zero(net, &net->gat[i], net->gat_floats)) fail = CERT_ERR_OOM;
        if (ok && fail == CERT_OK && !net->skip_from.empty()) {
            // a traversal that stops early may leave one more partial bound per row (the waiting coefficients)
            net->d_slots += 1;
            int ld_max = net->ld0;
            for (const LayerDev &L : net->layers) ld_max = std::max(ld_max, L.ld_out);
            if (!dev_alloc_zero(net, &net->zeros, (size_t)ld_max)) fail = CERT_ERR_OOM;
        }
        if (fail == CERT_OK &&
            (!dev_alloc_zero(net, &net->dbuf[0], (size_t)net->d_slots * max_rows) ||
             !dev_alloc_zero(net, &net->dbuf[1], (size_t)net->d_slots * max_rows)))
            fail = CERT_ERR_OOM;
    }
    if (fail == CERT_OK) {
        cert::convt_prepare();
        cert::conv_patch_prepare();
        if (cudaDeviceSynchronize() != cudaSuccess) fail = CERT_ERR_CUDA;
    }
    *partial = nullptr;
    if (fail != CERT_OK) {
        cudaGetLastError();
        free_net(net);
        return fail;
    }
    *out = net;
    return CERT_OK;
}

cert_status_t cert_net_create(const cert_layer_desc_t *layers, int n_layers, int max_batch, float clip_lo,
                              float clip_hi, cert_net_t **out) {
    return cert_net_create_residual(layers, n_layers, nullptr, max_batch, clip_lo, clip_hi, out);
}

cert_status_t cert_net_create_residual(const cert_layer_desc_t *layers, int n_layers, const int *skip_from,
                                       int max_batch, float clip_lo, float clip_hi, cert_net_t **out) {
    if (!out) return CERT_ERR_INVALID_ARG;
    *out = nullptr;
    // the set-up code builds host vectors: a failed host allocation must come back as a status, not cross the C ABI
    cert_net *partial = nullptr;
    try {
        return create_impl(layers, n_layers, skip_from, max_batch, clip_lo, clip_hi, out, &partial);
    } catch (const std::bad_alloc &) {
    } catch (...) {
        cudaGetLastError();
        if (partial) free_net(partial);
        *out = nullptr;
        return CERT_ERR_CUDA;
    }
    cudaGetLastError();
    if (partial) free_net(partial);
    *out = nullptr;
    return CERT_ERR_OOM;
}

cert_status_t cert_deeppoly_bounds(cert_net_t *net, const float *centers, float eps, int batch, float *lb_out,
                                   float *ub_out, void *stream) {
    return cert_backsub_bounds(net, centers, eps, batch, nullptr, lb_out, ub_out, stream);
}

cert_status_t cert_backsub_bounds(cert_net_t *net, const float *centers, float eps, int batch,
                                  const int *backsteps, float *lb_out, float *ub_out, void *stream) {
    return backsub_impl(net, centers, eps, batch, backsteps, lb_out, ub_out, static_cast<cudaStream_t>(stream), -1);
}

cert_status_t cert_deeppoly_bounds_host(cert_net_t *net, const float *centers_host, float eps, int batch,
                                        float *lb_host, float *ub_host, void *stream) {
    return cert_backsub_bounds_host(net, centers_host, eps, batch, nullptr, lb_host, ub_host, stream);
}

// The status code a non-zero status word stands for: a run-out wait first, then a refused store of the checking
// build, then an fp16 overflow.
static cert_status_t status_of_flag(int flag) {
    if (flag & 1) return CERT_ERR_TIMEOUT;
    if (flag & 4) return CERT_ERR_BOUNDS;
    if (flag & 2) return CERT_ERR_RANGE;
    return CERT_OK;
}

// Reads the sticky status word after the stream has drained; clears it when set.
static cert_status_t read_status(cert_net *net, cudaStream_t st, int *flag_out) {
    int flag = 0;
    if (cudaMemcpyAsync(&flag, net->status_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    if (flag != 0 && (cudaMemsetAsync(net->status_dev, 0, sizeof(int), st) != cudaSuccess ||
                      cudaStreamSynchronize(st) != cudaSuccess)) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    *flag_out = flag;
    return CERT_OK;
}

cert_status_t cert_backsub_bounds_host(cert_net_t *net, const float *centers_host, float eps, int batch,
                                       const int *backsteps, float *lb_host, float *ub_host, void *stream) {
    if (!net || !centers_host || !lb_host || !ub_host) return CERT_ERR_INVALID_ARG;
    if (batch < 1) return CERT_ERR_INVALID_ARG;
    if (batch > net->max_batch) return CERT_ERR_BATCH_TOO_LARGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    size_t in_bytes = (size_t)batch * net->n0 * sizeof(float);
    size_t out_bytes = (size_t)batch * net->n_total * sizeof(float);
    if (cudaMemcpyAsync(net->centers_dev, centers_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    // This call waits for its results anyway, so it also reads the device's status word: bounds that a run-out
    // wait or an fp16 overflow invalidated are never handed back as a success.  Under AUTO an overflow (which
    // the create-time range proof rules out; this is the second line of defence) re-runs the call in the TF32 split.
    int forced = -1;
    for (int attempt = 0; attempt < 2; ++attempt) {
        cert_status_t s = backsub_impl(net, net->centers_dev, eps, batch, backsteps, net->lb_dev, net->ub_dev, st, forced);
        if (s != CERT_OK) return s;
        if (cudaMemcpyAsync(lb_host, net->lb_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaMemcpyAsync(ub_host, net->ub_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
            cudaGetLastError();
            return CERT_ERR_CUDA;
        }
        int flag = 0;
        s = read_status(net, st, &flag);
        if (s != CERT_OK) return s;
        if (flag & 5) return status_of_flag(flag);
        if (flag & 2) {
            if (net->contraction == CERT_CONTRACTION_AUTO && attempt == 0 && net->tc_ok) {
                forced = CERT_CONTRACTION_TC3XTF32;
                continue;
            }
            return CERT_ERR_RANGE;
        }
        return CERT_OK;
    }
    return CERT_ERR_RANGE;
}

static cert_status_t enable_reusecert_impl(cert_net_t *net);

cert_status_t cert_net_enable_reusecert(cert_net_t *net) {
    try {
        return enable_reusecert_impl(net);
    } catch (const std::bad_alloc &) {
        cudaGetLastError();
        return CERT_ERR_OOM;        // what was allocated so far belongs to the net and goes with it
    } catch (...) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
}

static cert_status_t enable_reusecert_impl(cert_net_t *net) {
    if (!net) return CERT_ERR_INVALID_ARG;
    if (net->reuse.on) return CERT_OK;
    const int K = net->n_layers;
    // the fp16-split contraction only: it holds the stated tolerance on deep nets, where rounding compounds from
    // layer to layer (each layer's shapes are built from the rounded shapes below), and the TF32 split does not
    if (K < 2 || !net->tc16_ok || !net->skip_from.empty()) return CERT_ERR_UNSUPPORTED;
    for (int k = 0; k < K; ++k)
        if (net->layers[k].kind != CERT_LAYER_FC) return CERT_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != net->device) { cudaGetLastError(); return CERT_ERR_INVALID_ARG; }
    ReuseState &R = net->reuse;
    R.R = round_up(net->n0 + 1, 32);
    R.layers.assign(K, ReuseLayer());
    int ld_max = 0;
    for (int k = 0; k < K; ++k) {
        R.layers[k].ld_s = round_up(2 * net->layers[k].n_out, 32);
        ld_max = std::max(ld_max, R.layers[k].ld_s);
    }
    const long long m_max = (long long)net->max_batch * R.R;
    const size_t elems = (size_t)m_max * ld_max;       // floats per buffer: a raw result, or a pair of halves
    R.lo_off = elems;                                  // in halves: the lo part of a pair is the buffer's second half
    for (int p = 0; p < 3; ++p)
        if (!dev_alloc_zero(net, &R.X[p], elems)) return CERT_ERR_OOM;
    if (!dev_alloc_zero(net, &R.colsum, (size_t)(m_max / 32) * ld_max)) return CERT_ERR_OOM;
    std::vector<float> w, t0, b2, bias;
    std::vector<__half> h16, l16;
    for (int k = 0; k < K; ++k) {
        const LayerDev &L = net->layers[k];
        const size_t rows_pad = round_up(L.n_out, kPad);
        w.resize(rows_pad * L.ld_in);
        if (cudaMemcpy(w.data(), L.W, w.size() * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) {
            cudaGetLastError();
            return CERT_ERR_CUDA;
        }
        if (k == 0) {
            t0.assign((size_t)round_up(L.n_in, kPad) * L.ld_out, 0.0f);
            for (int t = 0; t < L.n_out; ++t)
                for (int s2 = 0; s2 < L.n_in; ++s2) t0[(size_t)s2 * L.ld_out + t] = w[(size_t)t * L.ld_in + s2];
            if (!dev_alloc(net, (void **)&R.W0t, t0.size() * sizeof(float))) return CERT_ERR_OOM;
            if (cudaMemcpy(R.W0t, t0.data(), t0.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
                return CERT_ERR_CUDA;
            continue;
        }
        ReuseLayer &RL = R.layers[k];
        const int n = L.n_out, m = L.n_in, ldb = R.layers[k - 1].ld_s;
        const size_t brows = round_up(2 * n, kPad);
        h16.assign(brows * ldb, __float2half_rn(0.0f));
        l16.assign(brows * ldb, __float2half_rn(0.0f));
        auto put16 = [&](int row, int col, float v) {
            const __half h = __float2half_rn(v);
            h16[(size_t)row * ldb + col] = h;
            l16[(size_t)row * ldb + col] = __float2half_rn((v - __half2float(h)) * cert::kLoScale);
        };
        for (int i = 0; i < n; ++i)
            for (int t = 0; t < m; ++t) {
                const float v = w[(size_t)i * L.ld_in + t];
                const float vp = v >= 0.0f ? v : 0.0f, vm = v >= 0.0f ? 0.0f : v;
                put16(i, t, vp);          // L_i takes L_t with W+ ...
                put16(i, m + t, vm);      // ... and U_t with W-
                put16(n + i, t, vm);      // U_i takes L_t with W- ...
                put16(n + i, m + t, vp);  // ... and U_t with W+
            }
        b2.assign(RL.ld_s, 0.0f);
        bias.resize(L.ld_out);
        if (cudaMemcpy(bias.data(), L.bias_n, bias.size() * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) {
            cudaGetLastError();
            return CERT_ERR_CUDA;
        }
        for (int i = 0; i < n; ++i) b2[i] = b2[n + i] = bias[i];
        if (!dev_alloc(net, (void **)&RL.B16_hi, h16.size() * sizeof(__half)) ||
            !dev_alloc(net, (void **)&RL.B16_lo, l16.size() * sizeof(__half)) ||
            !dev_alloc(net, (void **)&RL.bias2, b2.size() * sizeof(float)))
            return CERT_ERR_OOM;
        if (cudaMemcpy(RL.B16_hi, h16.data(), h16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(RL.B16_lo, l16.data(), l16.size() * sizeof(__half), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(RL.bias2, b2.data(), b2.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
            return CERT_ERR_CUDA;
        RL.plan16 = cert::tc16_tile_plan(2 * n);
        if (RL.plan16.stages < 2) return CERT_ERR_UNSUPPORTED;
        bool ok = cert::tc16_make_map(&RL.b16_hi, RL.B16_hi, 2 * m, 2 * n, ldb, 64, RL.plan16.bn / 2) &&
                  cert::tc16_make_map(&RL.b16_lo, RL.B16_lo, 2 * m, 2 * n, ldb, 64, RL.plan16.bn / 2);
        for (int p = 0; p < 3 && ok; ++p) {
            const __half *xh = reinterpret_cast<const __half *>(R.X[p]);
            ok = cert::tc16_make_map(&RL.a16_hi[p], xh, 2 * m, m_max, ldb, 64, 128) &&
                 cert::tc16_make_map(&RL.a16_lo[p], xh + R.lo_off, 2 * m, m_max, ldb, 64, 128) &&
                 cert::tc_make_map(&RL.o32[p], R.X[p], RL.ld_s, m_max, RL.ld_s, 32);
        }
        if (!ok) return CERT_ERR_CUDA;
    }
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CERT_ERR_CUDA; }
    R.on = true;
    return CERT_OK;
}

cert_status_t cert_reusecert_bounds(cert_net_t *net, const float *centers, float eps, int batch, float *lb_out,
                                    float *ub_out, void *stream) {
    if (!net || !centers || !lb_out || !ub_out) return CERT_ERR_INVALID_ARG;
    if (batch < 1 || !(eps >= 0.0f) || std::isinf(eps)) return CERT_ERR_INVALID_ARG;
    if (batch > net->max_batch) return CERT_ERR_BATCH_TOO_LARGE;
    if (!net->reuse.on) return CERT_ERR_UNSUPPORTED;
    // served in the fp16 split only (see cert_net_enable_reusecert): a net set to another mode is refused
    if (net->contraction != CERT_CONTRACTION_AUTO && net->contraction != CERT_CONTRACTION_TC3XFP16)
        return CERT_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ReuseState &R = net->reuse;
    const int K = net->n_layers, n_total = net->n_total;
    const long long rows = (long long)batch * R.R;
#ifdef CERT_BOUNDS
    {
        const void *extra[2] = {lb_out, ub_out};
        const size_t bytes[2] = {(size_t)batch * n_total * sizeof(float), (size_t)batch * n_total * sizeof(float)};
        const cert_status_t bs = bounds_sync(net, extra, bytes, 2);
        if (bs != CERT_OK) return bs;
    }
#endif
    Recorder rec(net, st);
    cert::launch_box(centers, eps, net->clip_lo, net->clip_hi, batch, net->n0, net->ld0, net->l0, net->u0, st);
    rec.mark(CERT_CLASS_INPUT);
    const LayerDev &L0 = net->layers[0];
    cert::launch_first_layer_bounds(L0, net->l0, net->u0, net->ld0, batch, lb_out, ub_out, n_total, st);
    rec.mark(CERT_CLASS_INPUT);
    cert::launch_relax(L0, lb_out, ub_out, n_total, batch, net->codes, net->n_relu, nullptr, 0, 0, st);
    rec.mark(CERT_CLASS_RELAX);
    // pair in X[xa], raw fp32 result in X[xb], scaled pair out in X[xc]
    auto hi_of = [&](int p) { return reinterpret_cast<__half *>(R.X[p]); };
    auto lo_of = [&](int p) { return reinterpret_cast<__half *>(R.X[p]) + R.lo_off; };
    int xa = 0, xb = 1, xc = 2;
    cert::launch_reuse_init16(R.W0t, L0.ld_out, L0, net->n0, R.R, R.layers[0].ld_s, rows, hi_of(xa), lo_of(xa),
                              net->status_dev, st);
    rec.mark(CERT_CLASS_RELU_STEP);
    for (int k = 1; k < K; ++k) {
        const LayerDev &Lk = net->layers[k];
        const ReuseLayer &RL = R.layers[k];
        cert::TcArgs a;
        std::memset(&a, 0, sizeof(a));
        a.M = rows; a.K = 2 * Lk.n_in; a.n_k = 1; a.ld_n = RL.ld_s;
        a.bn = RL.plan16.bn; a.n_tiles = RL.plan16.n_tiles; a.stages = RL.plan16.stages;
        a.tmem_cols = RL.plan16.tmem_cols;
        a.total_tiles = (int)cert::ceil_div_ll(rows, 256) * RL.plan16.n_tiles;
        a.l0 = net->l0; a.u0 = net->u0;
        a.reuse_R = R.R; a.reuse_n0 = net->n0; a.reuse_ld0 = net->ld0; a.n_half = Lk.n_out;
        a.bias2 = RL.bias2; a.colsum = R.colsum;
        a.status = net->status_dev;
        const int pairs = std::min(a.total_tiles, net->sm_count / 2);
        cert::launch_gemm_tc16(cert::TC_EPI_REUSE, false, pairs, RL.a16_hi[xa], RL.a16_lo[xa], RL.b16_hi, RL.b16_lo,
                               RL.o32[xb], RL.o32[xb], a, RL.plan16.smem_bytes, st);
        rec.mark(CERT_CLASS_AFFINE);
        cert::launch_reuse_relax(R.colsum, RL.ld_s, R.R / 32, Lk, batch, lb_out, ub_out, n_total, net->codes,
                                 net->n_relu, st);
        rec.mark(CERT_CLASS_RELAX);
        if (k + 1 < K) {
            cert::launch_reuse_scale16(R.X[xb], hi_of(xc), lo_of(xc), RL.ld_s, Lk, net->n0, R.R, rows, net->status_dev, st);
            rec.mark(CERT_CLASS_RELU_STEP);
        }
        const int t = xa; xa = xc; xc = xb; xb = t;
    }
    net->last_batch = batch;
    net->last_launches = rec.launches;
    net->last_paths = 2 | 4 | 16;
    net->prof_marks = rec.marks;
    if (cudaPeekAtLastError() != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}

cert_status_t cert_reusecert_bounds_host(cert_net_t *net, const float *centers_host, float eps, int batch,
                                         float *lb_host, float *ub_host, void *stream) {
    if (!net || !centers_host || !lb_host || !ub_host) return CERT_ERR_INVALID_ARG;
    if (batch < 1) return CERT_ERR_INVALID_ARG;
    if (batch > net->max_batch) return CERT_ERR_BATCH_TOO_LARGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    size_t in_bytes = (size_t)batch * net->n0 * sizeof(float);
    size_t out_bytes = (size_t)batch * net->n_total * sizeof(float);
    if (cudaMemcpyAsync(net->centers_dev, centers_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    cert_status_t s = cert_reusecert_bounds(net, net->centers_dev, eps, batch, net->lb_dev, net->ub_dev, stream);
    if (s != CERT_OK) return s;
    if (cudaMemcpyAsync(lb_host, net->lb_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(ub_host, net->ub_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    int flag = 0;
    s = read_status(net, st, &flag);
    if (s != CERT_OK) return s;
    return status_of_flag(flag);
}

cert_status_t cert_net_destroy(cert_net_t *net) {
    if (!net) return CERT_ERR_INVALID_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    free_net(net);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}

int cert_net_num_neurons(const cert_net_t *net) { return net ? net->n_total : -1; }
int cert_net_num_relu_neurons(const cert_net_t *net) { return net ? net->n_relu : -1; }

cert_status_t cert_net_branch_codes(cert_net_t *net, unsigned char *codes_out, void *stream) {
    if (!net) return CERT_ERR_INVALID_ARG;
    if (net->last_batch < 1) return CERT_ERR_INVALID_ARG;
    size_t bytes = (size_t)net->last_batch * net->n_relu;
    if (bytes == 0) return CERT_OK;
    if (!codes_out) return CERT_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(codes_out, net->codes, bytes, cudaMemcpyDeviceToDevice,
                        static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}

cert_status_t cert_net_last_status(cert_net_t *net, void *stream) {
    if (!net) return CERT_ERR_INVALID_ARG;
    int flag = 0;
    cert_status_t s = read_status(net, static_cast<cudaStream_t>(stream), &flag);
    if (s != CERT_OK) return s;
    return status_of_flag(flag);
}

int cert_net_check_guards(cert_net_t *net, void *stream) {
    if (!net) return -1;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { cudaGetLastError(); return -1; }
    unsigned char host[2 * kGuardBytes];
    for (size_t i = 0; i < net->guards.size(); ++i) {
        const cert_net::Guarded &g = net->guards[i];
        if (cudaMemcpy(host, g.base, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(host + kGuardBytes, g.base + kGuardBytes + g.bytes, kGuardBytes, cudaMemcpyDeviceToHost) !=
                cudaSuccess) {
            cudaGetLastError();
            return -1;
        }
        for (size_t b = 0; b < 2 * kGuardBytes; ++b)
            if (host[b] != kGuardByte) return (int)i + 1;
    }
    return 0;
}

int cert_built_with_checked_stores(void) {
#ifdef CERT_BOUNDS
    return 1;
#else
    return 0;
#endif
}

cert_status_t cert_net_selftest_checked_store(cert_net_t *net, void *stream) {
    if (!net) return CERT_ERR_INVALID_ARG;
#ifdef CERT_BOUNDS
    const cert_status_t bs = bounds_sync(net, nullptr, nullptr, 0);
    if (bs != CERT_OK) return bs;
    // one float past the end of the box array: inside the allocation's trailing guard, outside every buffer
    cert::launch_checked_store_selftest(net->l0 + (size_t)net->max_batch * net->ld0, static_cast<cudaStream_t>(stream));
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return CERT_ERR_CUDA; }
    return CERT_OK;
#else
    (void)stream;
    return CERT_ERR_UNSUPPORTED;
#endif
}

int cert_net_auto_contraction(const cert_net_t *net) {
    if (!net) return -1;
    if (net->auto_fp16) return CERT_CONTRACTION_TC3XFP16;
    return net->tc_ok ? CERT_CONTRACTION_TC3XTF32 : CERT_CONTRACTION_FFMA;
}

float cert_net_fp16_coefficient_bound(const cert_net_t *net, int layer) {
    if (!net || layer >= net->n_layers) return -1.0f;
    if (layer < 0) return net->fp16_coef_bound;
    return layer < (int)net->fp16_layer_bound.size() ? net->fp16_layer_bound[layer] : INFINITY;
}

cert_status_t cert_net_set_contraction(cert_net_t *net, int mode) {
    if (!net) return CERT_ERR_INVALID_ARG;
    if (mode != CERT_CONTRACTION_AUTO && mode != CERT_CONTRACTION_FFMA && mode != CERT_CONTRACTION_TC3XTF32 &&
        mode != CERT_CONTRACTION_TC3XFP16)
        return CERT_ERR_INVALID_ARG;
    if (mode == CERT_CONTRACTION_TC3XFP16 && !net->tc16_ok) return CERT_ERR_UNSUPPORTED;
    if (mode == CERT_CONTRACTION_TC3XTF32 && !net->tc_ok) return CERT_ERR_UNSUPPORTED;
    net->contraction = mode;
    return CERT_OK;
}

cert_status_t cert_net_selftest_bounded_wait(cert_net_t *net, void *stream) {
    if (!net) return CERT_ERR_INVALID_ARG;
    cert::launch_bounded_wait_selftest(net->status_dev, static_cast<cudaStream_t>(stream));
    if (cudaPeekAtLastError() != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}

cert_status_t cert_net_set_profiling(cert_net_t *net, int on) {
    if (!net) return CERT_ERR_INVALID_ARG;
    if (on && net->prof_events.empty()) {
        // one event per launch of the longest schedule, plus the opening one
        int K = net->n_layers;
        int n = 4 + 2 * K + K * (K + 1) + 8;
        net->prof_events.resize(n);
        net->prof_class.assign(n, 0);
        for (int i = 0; i < n; ++i)
            if (cudaEventCreate(&net->prof_events[i]) != cudaSuccess) {
                cudaGetLastError();
                for (int j = 0; j < i; ++j) cudaEventDestroy(net->prof_events[j]);
                net->prof_events.clear();
                return CERT_ERR_CUDA;
            }
    }
    net->profiling = on != 0;
    net->prof_marks = 0;
    return CERT_OK;
}

cert_status_t cert_net_profile(cert_net_t *net, float *ms_out, int *launches_out) {
    if (!net || !ms_out || !launches_out) return CERT_ERR_INVALID_ARG;
    for (int c = 0; c < CERT_N_CLASSES; ++c) { ms_out[c] = 0.0f; launches_out[c] = 0; }
    if (net->prof_marks == 0) return CERT_OK;
    if (cudaEventSynchronize(net->prof_events[net->prof_marks]) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    for (int i = 0; i < net->prof_marks; ++i) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, net->prof_events[i], net->prof_events[i + 1]) != cudaSuccess) {
            cudaGetLastError();
            return CERT_ERR_CUDA;
        }
        ms_out[net->prof_class[i]] += ms;
        launches_out[net->prof_class[i]] += 1;
    }
    return CERT_OK;
}

int cert_net_last_contraction_paths(const cert_net_t *net) { return net ? net->last_paths : -1; }

cert_status_t cert_net_set_conv_patches(cert_net_t *net, int on) {
    if (!net) return CERT_ERR_INVALID_ARG;
    if (on && !net->skip_from.empty()) return CERT_ERR_UNSUPPORTED;   // rows of such nets stay dense
    net->conv_patches = on != 0;
    return CERT_OK;
}

int cert_net_last_launch_count(const cert_net_t *net) { return net ? net->last_launches : -1; }

double cert_net_backstep_flops(const cert_net_t *net, int batch) {
    if (!net || batch < 1) return 0.0;
    double f = 0.0;
    for (int k = 1; k < net->n_layers; ++k) {
        double rows = 2.0 * batch * net->layers[k].n_out;
        for (int j = 0; j < k; ++j) {
            const LayerDev &L = net->layers[j];
            double per_row = L.kind == CERT_LAYER_FC
                                 ? 2.0 * L.n_out * L.n_in
                                 : 2.0 * L.n_out * (double)L.c_in * L.kh * L.kw;
            f += rows * per_row;
        }
    }
    return f;
}

}  // extern "C"
