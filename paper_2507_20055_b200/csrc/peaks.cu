// Micro-kernels that measure the denominators of the contraction rooflines on the device at hand: the rate of
// tcgen05.mma kind::f16 and kind::tf32 in the instruction shape the product kernels use (CTA pairs, 256 x 256
// tiles, both operands resident in shared memory, no loads in the loop), and the rate of the fp32 FMA units on
// a register-only loop; and the rate at which the SMs take bulk copies from L2 into shared memory, which is what
// bounds the fp16-split contraction once its operands are staged more than once.  (No counterpart in the paper:
// measurement support.)
//
// Each kernel also reads the SM cycle counter and the global nanosecond timer at its start and end, so that the
// rate comes with the SM clock it was measured at (rates are compared per cycle, whatever the power state).
#include <cmath>

#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "gemm_tc16.cuh"
#include "tc_ptx.cuh"

namespace cert {

namespace {

constexpr int kPeakBM = 128;           // rows per CTA of the pair
constexpr int kPeakBN = 256;           // columns of the tile
constexpr int kTileBytes = 128 * 128;  // 128 rows of 128 bytes: one K-major swizzle-128 operand tile

struct __align__(8) PeakBars {
    uint64_t done[2];
    uint32_t tmem_base;
    uint32_t pad;
};

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// A value in [-1, 1) from a counter (the operands only have to be ordinary numbers: zeros would understate the
// power the tensor cores draw, and with it overstate the clock).
__device__ __forceinline__ float hash_unit(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return (float)(int)(x >> 8) * (1.0f / 8388608.0f) - 1.0f;
}

// KIND 0: kind::f16 (K = 16 per instruction), KIND 1: kind::tf32 (K = 8).  One CTA pair per cluster; the leader
// issues `n_mma` instructions in groups of `burst`, each group followed by a commit and a bounded wait.
template <int KIND>
__global__ void __launch_bounds__(128, 1)
mma_peak_kernel(int n_mma, int burst, int *status, unsigned long long *clocks_out) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *tile_a = smem, *tile_b = smem + kTileBytes;
    PeakBars *bars = reinterpret_cast<PeakBars *>(smem + 2 * kTileBytes);
    const uint32_t rank = cluster_ctarank();
    const int warp = threadIdx.x >> 5;
    // operand tiles: every byte position of the two tiles gets a value (the swizzle only permutes positions)
    if (KIND == 0) {
        __half *h = reinterpret_cast<__half *>(smem);
        for (int i = threadIdx.x; i < 2 * kTileBytes / 2; i += blockDim.x)
            h[i] = __float2half_rn(hash_unit((uint32_t)i * 2654435761u + blockIdx.x));
    } else {
        float *f = reinterpret_cast<float *>(smem);
        for (int i = threadIdx.x; i < 2 * kTileBytes / 4; i += blockDim.x)
            f[i] = tf32_round(hash_unit((uint32_t)i * 2654435761u + blockIdx.x));
    }
    if (threadIdx.x == 0) {
        mbar_init(&bars->done[0], 1);
        mbar_init(&bars->done[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&bars->tmem_base)), "r"((uint32_t)kPeakBN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    unsigned long long c0 = 0, t0 = 0;
    if (threadIdx.x == 0 && rank == 0) {
        c0 = (unsigned long long)clock64();
        t0 = global_ns();
        uint32_t idesc = ((uint32_t)(kPeakBN >> 3) << 17) | ((uint32_t)((kPeakBM * 2) >> 4) << 24) | (1u << 4);
        if (KIND == 1) idesc |= (2u << 7) | (2u << 10);
        const uint64_t da = make_desc(smem_u32(tile_a)), db = make_desc(smem_u32(tile_b));
        // bursts alternate between two barriers: a burst is committed, then the one before it is waited for, so
        // that the tensor pipe always has work queued
        uint32_t phase[2] = {0, 0};
        bool ok = true;
        int b = 0;
        for (int done = 0; done < n_mma && ok; done += burst, ++b) {
            const int n = n_mma - done < burst ? n_mma - done : burst;
            for (int i = 0; i < n; ++i) {
                const uint64_t ko = (uint64_t)((i & 3) * 2);        // the four 32-byte k-steps of the 128-byte rows
                if (KIND == 0) mma_f16<2>(tmem_base, da + ko, db + ko, idesc, (done | i) ? 1u : 0u);
                else mma_tf32<2>(tmem_base, da + ko, db + ko, idesc, (done | i) ? 1u : 0u);
            }
            tcgen05_commit<2>(&bars->done[b & 1]);
            if (b > 0) {
                ok = mbar_wait(&bars->done[(b - 1) & 1], phase[(b - 1) & 1]);
                phase[(b - 1) & 1] ^= 1;
            }
        }
        if (ok && b > 0) ok = mbar_wait(&bars->done[(b - 1) & 1], phase[(b - 1) & 1]);
        if (!ok) atomicOr(status, 1);
        if (blockIdx.x == 0) {
            clocks_out[0] = (unsigned long long)clock64() - c0;
            clocks_out[1] = global_ns() - t0;
        }
    }
    // (the commits are multicast to the peer's barriers too; nobody waits there, and the peer stays until the
    // cluster barrier below, which the leader reaches only when every instruction has retired)
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kPeakBN)
                     : "memory");
    }
}

// Eight independent chains of fused multiply-adds per thread, all in registers.
__global__ void __launch_bounds__(1024, 1)
ffma_peak_kernel(int iters, float *sink, unsigned long long *clocks_out) {
    float a[8], x = 1.0f + 1e-7f * (float)threadIdx.x, y = 1e-3f * (float)(blockIdx.x + 1);
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = (float)i;
    unsigned long long c0 = 0, t0 = 0;
    if (threadIdx.x == 0 && blockIdx.x == 0) { c0 = (unsigned long long)clock64(); t0 = global_ns(); }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] = fmaf(a[i], x, y);
    }
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += a[i];
    if (s == 12345.678f) sink[0] = s;                 // keeps the chains alive
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        clocks_out[0] = (unsigned long long)clock64() - c0;
        clocks_out[1] = global_ns() - t0;
    }
}

// KIND 3: what the SMs take in from L2 through TMA tile loads into shared memory, the path the contractions' operand
// tiles travel.  One CTA per SM (it asks for most of the shared memory) keeps eight 16 KB tile loads in flight from
// a region of its own of a buffer that fits L2 (the tiles of a 128-row panel of a 1024-wide fp16 matrix, over and
// over), and nothing reads what lands: the rate is the intake alone.  A single thread issues and waits (bounded waits; on a run-out it stops issuing and waits for what is
// in flight before the CTA gives its shared memory back).
constexpr int kIntakeSlots = 8;
constexpr int kIntakeChunk = 16 * 1024;             // the size of an operand tile of the fp16-split kernel
constexpr int kIntakeTilesPerRow = 16;              // the block's region: 128 rows of 16 x 64 halves (2 KB pitch, 256 KB)

struct __align__(8) IntakeBars {
    uint64_t full[kIntakeSlots];
};

__global__ void __launch_bounds__(128, 1)
l2_intake_kernel(const __grid_constant__ CUtensorMap map, int n_loads, int *status, unsigned long long *clocks_out) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    IntakeBars *bars = reinterpret_cast<IntakeBars *>(smem + kIntakeSlots * kIntakeChunk);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kIntakeSlots; ++s) mbar_init(&bars->full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long c0 = (unsigned long long)clock64(), t0 = global_ns();
        bool ok = true;
        int issued = 0;
        for (int i = 0; i < n_loads && ok; ++i) {
            const int s = i % kIntakeSlots;
            const int use = i / kIntakeSlots;
            if (use > 0 && !mbar_wait(&bars->full[s], (uint32_t)((use - 1) & 1))) { ok = false; break; }
            mbar_arrive_expect_tx(&bars->full[s], kIntakeChunk);
            // tile i of the block's 128 rows: 64 halves (one 128-byte swizzle row) x 128 rows, as an A tile of the
            // fp16-split contraction
            tma_load_2d<1>(smem_u32(smem + (size_t)s * kIntakeChunk), &map, smem_u32(&bars->full[s]),
                           (i % kIntakeTilesPerRow) * 64, (int)blockIdx.x * 128);
            issued = i + 1;
        }
        // everything in flight lands before the CTA ends
        const int first = issued > kIntakeSlots ? issued - kIntakeSlots : 0;
        for (int i = first; i < issued; ++i)
            if (!mbar_wait(&bars->full[i % kIntakeSlots], (uint32_t)((i / kIntakeSlots) & 1))) ok = false;
        if (!ok) atomicOr(status, 1);
        if (blockIdx.x == 0) {
            clocks_out[0] = (unsigned long long)clock64() - c0;
            clocks_out[1] = global_ns() - t0;
        }
    }
    __syncthreads();
}

}  // namespace

}  // namespace cert

extern "C" cert_status_t cert_peak_microbench(int kind, double target_ms, double *tflops_out, double *sm_mhz_out,
                                              double *ms_out, void *stream) {
    using namespace cert;
    if (kind < 0 || kind > 3 || !tflops_out || !(target_ms > 0.0) || target_ms > 2000.0) return CERT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2) {
        cudaGetLastError();
        return CERT_ERR_CUDA;
    }
    int *status = nullptr;
    unsigned long long *clocks = nullptr;
    float *sink = nullptr;
    uint8_t *l2buf = nullptr;
    const unsigned long long intake_per_cta = 256ull * 1024ull;     // 128 rows of 2 KB; 148 SMs: 37 MB, inside the 126 MB L2
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cert_status_t rc = CERT_OK;
    auto cleanup = [&]() {
        if (status) cudaFree(status);
        if (clocks) cudaFree(clocks);
        if (sink) cudaFree(sink);
        if (l2buf) cudaFree(l2buf);
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
    };
    if (cudaMalloc(reinterpret_cast<void **>(&status), sizeof(int)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void **>(&clocks), 2 * sizeof(unsigned long long)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void **>(&sink), sizeof(float)) != cudaSuccess ||
        cudaMemset(status, 0, sizeof(int)) != cudaSuccess ||
        cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_OOM;
    }
    if (kind == 3 && (cudaMalloc(reinterpret_cast<void **>(&l2buf), (size_t)sms * intake_per_cta) != cudaSuccess ||
                      cudaMemsetAsync(l2buf, 0x3c, (size_t)sms * intake_per_cta, st) != cudaSuccess)) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_OOM;
    }
    TcMap intake_map;
    if (kind == 3 && (!tc16_prepare_kernels() ||
                      !tc16_make_map(&intake_map, reinterpret_cast<const __half *>(l2buf), 64 * kIntakeTilesPerRow,
                                     (long long)sms * 128, 64 * kIntakeTilesPerRow, 64, 128))) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_UNSUPPORTED;
    }
    // The kernel needs 34 KB, but it asks for 200 KB so that a multiprocessor holds exactly one of its CTAs, as
    // with the product kernels: two CTAs on one SM would compete for its tensor memory (an allocation that
    // cannot be served blocks without a limit), and a CTA pair must sit on two SMs.
    const int smem = 200 * 1024;
    static_assert(2 * kTileBytes + 1024 + (int)sizeof(PeakBars) <= 200 * 1024, "operand tiles fit");
    static_assert(kIntakeSlots * kIntakeChunk + 1024 + (int)sizeof(IntakeBars) <= 200 * 1024, "intake ring fits");
    const int pairs = sms / 2;
    double flop_per_unit = 0.0;      // per MMA instruction of one pair, or per loop iteration of the whole grid
    if (kind == 0) flop_per_unit = 2.0 * (kPeakBM * 2) * kPeakBN * 16;
    if (kind == 1) flop_per_unit = 2.0 * (kPeakBM * 2) * kPeakBN * 8;
    const int ffma_blocks = sms;
    if (kind == 2) flop_per_unit = 2.0 * 32.0 * 1024.0 * ffma_blocks;
    if (kind == 3) flop_per_unit = (double)kIntakeChunk * sms;          // bytes per copy of every CTA
    if (kind == 3 && cudaFuncSetAttribute(l2_intake_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_CUDA;
    }
    if (kind < 2 &&
        (cudaFuncSetAttribute(mma_peak_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
         cudaFuncSetAttribute(mma_peak_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)) {
        cudaGetLastError();
        cleanup();
        return CERT_ERR_CUDA;
    }
    auto launch = [&](int units) {
        if (kind == 2) {
            ffma_peak_kernel<<<ffma_blocks, 1024, 0, st>>>(units, sink, clocks);
            return;
        }
        if (kind == 3) {
            l2_intake_kernel<<<sms, 128, smem, st>>>(reinterpret_cast<const CUtensorMap &>(intake_map), units, status, clocks);
            return;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(pairs * 2), 1, 1);
        cfg.blockDim = dim3(128, 1, 1);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const int burst = 256;
        if (kind == 0) cudaLaunchKernelEx(&cfg, mma_peak_kernel<0>, units, burst, status, clocks);
        else cudaLaunchKernelEx(&cfg, mma_peak_kernel<1>, units, burst, status, clocks);
    };
    // a short calibration run sizes the timed one for about target_ms
    int units = kind == 2 ? 2000 : 4096;
    float ms = 0.0f;
    for (int pass = 0; pass < 2 && rc == CERT_OK; ++pass) {
        if (cudaEventRecord(e0, st) != cudaSuccess) { rc = CERT_ERR_CUDA; break; }
        launch(units);
        if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
            cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
            rc = CERT_ERR_CUDA;
            break;
        }
        if (pass == 0) {
            double scaled = (double)units * target_ms / (ms > 1e-3f ? ms : 1e-3f);
            if (scaled > 5e7) scaled = 5e7;
            if (scaled < 64) scaled = 64;
            units = (int)scaled;
        }
    }
    int flag = 0;
    unsigned long long host_clocks[2] = {0, 0};
    if (rc == CERT_OK && (cudaMemcpy(&flag, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
                          cudaMemcpy(host_clocks, clocks, sizeof(host_clocks), cudaMemcpyDeviceToHost) != cudaSuccess))
        rc = CERT_ERR_CUDA;
    if (rc == CERT_OK && flag) rc = CERT_ERR_TIMEOUT;
    if (rc == CERT_OK) {
        const double total = kind >= 2 ? flop_per_unit * units : flop_per_unit * units * pairs;
        *tflops_out = total / ((double)ms * 1e-3) / 1e12;
        if (sm_mhz_out) *sm_mhz_out = host_clocks[1] ? (double)host_clocks[0] * 1e3 / (double)host_clocks[1] : 0.0;
        if (ms_out) *ms_out = ms;
    } else {
        cudaGetLastError();
    }
    cleanup();
    return rc;
}
