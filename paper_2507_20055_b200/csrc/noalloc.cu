// Interval bounds of one FC layer over a batch of boxes, for callers that must
// not allocate device memory.  The box endpoints that the regular path keeps
// in the net's workspace live here in a fixed array inside the library image.
#include <cmath>
#include <mutex>

#include "common.cuh"

namespace {

// Room for batch * round_up(in_features, 32) floats per endpoint array.
constexpr size_t kNoAllocMaxFloats = size_t(1) << 20;   // 4 MiB each, 8 MiB in total

// Lower endpoints in the first half, upper endpoints in the second.  Every GPU
// that loads the library carries these 8 MiB until the process exits.
static __device__ __align__(256) float g_box_scratch[2 * kNoAllocMaxFloats];

constexpr int kMaxDevices = 64;
float *g_scratch_addr[kMaxDevices] = {};   // device address of g_box_scratch, per device
std::mutex g_scratch_mutex;

// In host code `g_box_scratch` is only a handle for the runtime, not a device
// pointer; the address the kernels need is looked up once per device, with
// that device current.
cert_status_t scratch_for_current_device(float **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices) return CERT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        float *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_box_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return CERT_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return CERT_OK;
}

}  // namespace

extern "C" cert_status_t cert_first_layer_bounds_noalloc(const float *weight, const float *bias,
                                                         int out_features, int in_features,
                                                         const float *centers, float eps, float clip_lo,
                                                         float clip_hi, int batch, float *lb_out,
                                                         float *ub_out, void *stream) {
    if (!weight || !bias || !centers || !lb_out || !ub_out) return CERT_ERR_INVALID_ARG;
    if (out_features < 1 || in_features < 1 || batch < 1) return CERT_ERR_INVALID_ARG;
    if (!(eps >= 0.0f) || std::isinf(eps)) return CERT_ERR_INVALID_ARG;
    if (std::isnan(clip_lo) || std::isnan(clip_hi) || clip_lo > clip_hi) return CERT_ERR_INVALID_ARG;
    const int ld0 = cert::round_up(in_features, cert::kPad);
    if ((size_t)batch * (size_t)ld0 > kNoAllocMaxFloats) return CERT_ERR_BATCH_TOO_LARGE;
    // one warp per (box, neuron), eight warps per block: the grid's x extent must hold them all
    if ((long long)batch * out_features > 8LL * 0x7FFFFFFF) return CERT_ERR_UNSUPPORTED;

    float *scratch = nullptr;
    cert_status_t s = scratch_for_current_device(&scratch);
    if (s != CERT_OK) return s;
    float *l0 = scratch, *u0 = scratch + kNoAllocMaxFloats;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
#ifdef CERT_BOUNDS
    {
        // checking build: what this call may write is the scratch array and the caller's two outputs
        static cert::BoundsTable t;
        t.n = 3;
        t.status = nullptr;
        t.lo[0] = (unsigned long long)scratch;
        t.hi[0] = t.lo[0] + 2 * kNoAllocMaxFloats * sizeof(float);
        t.lo[1] = (unsigned long long)lb_out;
        t.hi[1] = t.lo[1] + (size_t)batch * out_features * sizeof(float);
        t.lo[2] = (unsigned long long)ub_out;
        t.hi[2] = t.lo[2] + (size_t)batch * out_features * sizeof(float);
        cert::bounds_upload_all(&t);
    }
#endif
    // The box kernel writes every element of [batch][ld0], padding included, so
    // nothing depends on what an earlier call left in the array.
    cert::launch_box(centers, eps, clip_lo, clip_hi, batch, in_features, ld0, l0, u0, st);
    cert::LayerDev L = {};
    L.kind = CERT_LAYER_FC;
    L.n_in = in_features;
    L.ld_in = in_features;        // the caller's weight rows are not padded
    L.n_out = out_features;
    L.ld_out = out_features;
    L.W = const_cast<float *>(weight);
    L.bias_n = const_cast<float *>(bias);
    L.out_off = 0;
    cert::launch_first_layer_bounds(L, l0, u0, ld0, batch, lb_out, ub_out, out_features, st);
    if (cudaPeekAtLastError() != cudaSuccess) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    return CERT_OK;
}
