// The whole traversal of an FC layer's expressions in one kernel (narrow FC nets, fp16-split form).
//
// For a layer k whose lower layers are at most 256 neurons wide, a 128-row panel of the coefficient
// matrix fits in shared memory as an fp16 pair.  A CTA pair then takes a 256-row panel through the
// entire while-loop of the traversal (Section 4.3: per iteration P = Q * W_j, then the clamp form of
// replace_lower/upper through the ReLU below) without the matrix ever leaving the chip:
//
//   start:   Q = rows of W_k through the ReLU of layer k-1, written straight into shared memory
//            in the swizzled K-major layout the tensor cores read;
//   step j:  P = Q * W_j on the tensor cores (W_j streamed through a TMA pipeline, accumulator in tensor
//            memory, one pass or two as in gemm_tc16.cu), the epilogue applies the ReLU back-step and
//            writes the result over Q as the next step's operand;
//   end:     the last step's epilogue is map(simplify_lower/upper) against the box (or the stored
//            bounds of the layer reached); only the bounds leave the kernel.
//
// A row's constant lives in registers of its owner threads (one per column group) for the whole
// traversal and leaves as kChainColGroups slots, summed by the next kernel: fixed order, no atomics.
// Warp roles: warp 0 = TMA producer of W_j tiles, warp 1 = MMA issuer (leader CTA) and TMEM owner,
// warps 2..17 = epilogue (kChainColGroups per TMEM lane quarter, each taking every kChainColGroups-th
// 32-column chunk; a step's MMAs and its epilogue cannot overlap, so the epilogue is spread wide).
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "gemm_tc16.cuh"
#include "chain16.cuh"
#include "tc_ptx.cuh"

namespace cert {

namespace {

constexpr int BM = 128;                          // rows per CTA
constexpr int BKH = 64;                          // halves of K per block: one 128-byte swizzle row
constexpr int kEpiWarps = 4 * kChainColGroups;   // kChainColGroups warps per TMEM lane quarter
constexpr int kThreadsChain = 64 + kEpiWarps * 32;
constexpr int kABlockBytes = BM * BKH * 2;       // one 64-column block of the panel (hi or lo): 16 KiB
constexpr int kAccCols = 256;                    // tensor-memory columns per accumulator
constexpr int CTAS = 2;
constexpr int kBlockWriters = 2 * 4;             // warps of a CTA that write a 64-column block: two chunks x four lane quarters

struct __align__(8) BarriersChain {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t a_ready[4];        // 64-column block kb of the panel in shared memory is complete (the epilogue warps of
                                // both CTAs that write its two 32-column chunks arrive): a step's first MMAs start
                                // on the blocks that are rewritten first while the epilogue still works on the rest
    uint64_t vec_full[2];       // a step's relaxation / bias vectors have landed in staging buffer 0 / 1
    uint64_t vec_empty[2];      // ... and every epilogue warp is done reading them
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait with cluster-scope acquire: what the peer CTA wrote before it arrived is visible after it.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((unsigned long long)(clock64() - t0) > kWaitCycles) return false;
    }
    return true;
}

// Plain (untiled) bulk copy global -> this CTA's shared memory; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Writes 32 consecutive columns [c0, c0+32) of panel row `row` as an fp16 pair into the K-major,
// 128-byte-swizzled blocks the MMA reads (block = c0 / 64; 16-byte chunk g of a row sits at g ^ (row & 7)).
__device__ __forceinline__ void write_panel_chunk(uint32_t a_hi, uint32_t a_lo, int row, int c0, const float (&q)[32],
                                                  bool check, bool &out_of_range, float lo_scale) {
    const uint32_t off = (uint32_t)(c0 >> 6) * kABlockBytes + (uint32_t)row * 128u;
    const int g0 = (c0 & 63) >> 3;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            __half h[2], l[2];
#pragma unroll
            for (int z = 0; z < 2; ++z) {
                const float x = q[g * 8 + e + z];
                out_of_range |= check && !(fabsf(x) <= 60000.0f);
                h[z] = __float2half_rn(x);
                l[z] = __float2half_rn((x - __half2float(h[z])) * lo_scale);
            }
            ph[e >> 1] = (uint32_t)__half_as_ushort(h[0]) | ((uint32_t)__half_as_ushort(h[1]) << 16);
            pl[e >> 1] = (uint32_t)__half_as_ushort(l[0]) | ((uint32_t)__half_as_ushort(l[1]) << 16);
        }
        const uint32_t sw = (uint32_t)(((g0 + g) ^ (row & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_hi + off + sw), "r"(ph[0]), "r"(ph[1]),
                     "r"(ph[2]), "r"(ph[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_lo + off + sw), "r"(pl[0]), "r"(pl[1]),
                     "r"(pl[2]), "r"(pl[3]) : "memory");
    }
}

template <bool ONEPASS>
__global__ void __launch_bounds__(kThreadsChain, 1)
chain16_kernel(const __grid_constant__ ChainParams P, const ChainArgs a) {
    // ONEPASS: see ChainArgs::one_pass (a template parameter so that the two-pass form carries none of its factors)
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *A_hi = smem;
    uint8_t *A_lo = smem + (size_t)a.a_blocks * kABlockBytes;
    uint8_t *Bst = smem + 2 * (size_t)a.a_blocks * kABlockBytes;
    const int stages = a.stages;
    const int kBChunkBytes = a.b_chunk_bytes, kStageBytes = 2 * a.b_chunk_bytes;
    float *vec_stage = reinterpret_cast<float *>(Bst + (size_t)stages * kStageBytes);
    const int vec_floats = 7 * a.vec_ld;
    BarriersChain *bars = reinterpret_cast<BarriersChain *>(reinterpret_cast<uint8_t *>(vec_stage) +
                                                            2 * (size_t)vec_floats * sizeof(float));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int group = (int)cluster_id_x();
    const int n_groups = (int)num_clusters_x();
    const long long n_panels = (a.M + BM * CTAS - 1) / (BM * CTAS);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->acc_full[i], 1);
            mbar_init(&bars->acc_empty[i], kEpiWarps * CTAS);
        }
        for (int i = 0; i < 4; ++i) mbar_init(&bars->a_ready[i], kBlockWriters * CTAS);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->vec_full[i], 1);
            mbar_init(&bars->vec_empty[i], kEpiWarps);
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&bars->tmem_base)),
                     "r"((uint32_t)(2 * kAccCols))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();      // the peer's barriers exist before anything arrives on them
    tcgen05_fence_after();
    pdl_wait();              // everything above needed nothing from the kernel before
    const uint32_t tmem_base = bars->tmem_base;
    volatile uint32_t *abort_flag = &bars->abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer: W_j tiles, step after step
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            int armed = 0;
            int vstep = 0;      // steps whose vectors were staged so far (buffer = vstep & 1)
            for (long long p = group; p < n_panels && ok; p += n_groups) {
                // boxes of this CTA's 128 rows: the first two are staged
                const long long row0 = p * (BM * CTAS) + (long long)rank * BM;
                const long long last_row = (row0 + BM - 1 < a.M ? row0 + BM - 1 : a.M - 1);
                const int b_last = (int)(last_row / (2LL * a.n_k));
                int b_first = (int)(row0 / (2LL * a.n_k));
                if (b_first > b_last) b_first = b_last;
                const int nb = b_last - b_first + 1 < 2 ? b_last - b_first + 1 : 2;
                for (int j = a.k - 1; j >= a.j_end && ok; --j) {
                    const ChainLayer &L = P.layer[j];
                    if (a.vec_ld > 0 && j > a.j_end) {
                        // the vectors the epilogue of this step reads: bias of the layer below, then per box lamL, lamU, nuU
                        const int buf = vstep & 1;
                        if (!mbar_wait(&bars->vec_empty[buf], ((vstep >> 1) & 1) ^ 1) || *abort_flag) { ok = false; break; }
                        float *dst = vec_stage + (size_t)buf * vec_floats;
                        const uint32_t bytes = (uint32_t)L.ld_in * sizeof(float);
                        const uint32_t n_copies = 1u + (L.relu_below ? 3u * (uint32_t)nb : 0u);
                        mbar_arrive_expect_tx(&bars->vec_full[buf], n_copies * bytes);
                        const uint32_t vbar = smem_u32(&bars->vec_full[buf]);
                        bulk_load(smem_u32(dst), L.bias_below, bytes, vbar);
                        if (L.relu_below)
                            for (int q = 0; q < nb; ++q) {
                                const size_t off = (size_t)(b_first + q) * L.ld_in;
                                float *d3 = dst + a.vec_ld + (size_t)q * 3 * a.vec_ld;
                                bulk_load(smem_u32(d3), L.lamL + off, bytes, vbar);
                                bulk_load(smem_u32(d3 + a.vec_ld), L.lamU + off, bytes, vbar);
                                bulk_load(smem_u32(d3 + 2 * a.vec_ld), L.nuU + off, bytes, vbar);
                            }
                        ++vstep;
                    }
                    const CUtensorMap *mh = reinterpret_cast<const CUtensorMap *>(&P.b_hi[j]);
                    const CUtensorMap *ml = reinterpret_cast<const CUtensorMap *>(&P.b_lo[j]);
                    const int num_kb = (L.n_out + BKH - 1) / BKH;
                    const int BNL = L.bn / CTAS;
                    const uint32_t b_bytes = (uint32_t)BNL * BKH * 2;
                    for (int nt = 0; nt < L.n_tiles && ok; ++nt) {
                        const int col0 = nt * L.bn + (int)rank * BNL;
                        // pass 1: the hi and lo tiles of a k-block per stage
                        for (int kb = 0; kb < num_kb; ++kb) {
                            if (!mbar_wait(&bars->empty[s], phase ^ 1) || *abort_flag) { ok = false; break; }
                            uint8_t *st = Bst + (size_t)s * kStageBytes;
                            if (rank == 0) mbar_arrive_expect_tx(&bars->full[s], 2 * b_bytes * CTAS);
                            const uint32_t bar = map_to_cta(smem_u32(&bars->full[s]), 0);
                            tma_load_2d<CTAS>(smem_u32(st), mh, bar, kb * BKH, col0);
                            tma_load_2d<CTAS>(smem_u32(st + kBChunkBytes), ml, bar, kb * BKH, col0);
                            ++armed;
                            if (++s == stages) { s = 0; phase ^= 1; }
                        }
                        // pass 2: the hi tiles of two k-blocks per stage
                        for (int kb = 0; !ONEPASS && kb < num_kb && ok; kb += 2) {
                            if (!mbar_wait(&bars->empty[s], phase ^ 1) || *abort_flag) { ok = false; break; }
                            uint8_t *st = Bst + (size_t)s * kStageBytes;
                            const bool two = kb + 1 < num_kb;
                            if (rank == 0) mbar_arrive_expect_tx(&bars->full[s], (two ? 2 : 1) * b_bytes * CTAS);
                            const uint32_t bar = map_to_cta(smem_u32(&bars->full[s]), 0);
                            tma_load_2d<CTAS>(smem_u32(st), mh, bar, kb * BKH, col0);
                            if (two) tma_load_2d<CTAS>(smem_u32(st + kBChunkBytes), mh, bar, (kb + 1) * BKH, col0);
                            ++armed;
                            if (++s == stages) { s = 0; phase ^= 1; }
                        }
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicOr(a.status, 1);
                if (rank == 0) {
                    // let the copies already in flight land before the CTA gives its shared memory back
                    int back = armed < stages ? armed : stages;
                    int ss = s;
                    uint32_t ph = phase;
                    for (int i = 0; i < back; ++i) {
                        if (--ss < 0) { ss = stages - 1; ph ^= 1; }
                        mbar_wait(&bars->full[ss], ph);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (the leader CTA)
        if (lane == 0 && rank == 0) {
            int s = 0;
            uint32_t phase = 0, a_phase = 0;      // a_phase: bit kb = phase of a_ready[kb]
            bool ok = true;
            int lt = 0;
            const uint32_t a_hi0 = smem_u32(A_hi), a_lo0 = smem_u32(A_lo);
            for (long long p = group; p < n_panels && ok; p += n_groups) {
                for (int j = a.k - 1; j >= a.j_end && ok; --j) {
                    const ChainLayer &L = P.layer[j];
                    const int num_kb = (L.n_out + BKH - 1) / BKH;
                    const int ksteps = (L.n_out + 15) / 16;       // 16-column MMA steps that hold neurons; the rest of the last block is zero
                    // (the panel over layer j's neurons arrives in shared memory block by block, in both CTAs)
                    // kind::f16: D = f32, A = B = f16 (format 0), both K-major
                    const uint32_t idesc = (1u << 4) | ((uint32_t)(L.bn >> 3) << 17) | ((uint32_t)((BM * CTAS) >> 4) << 24);
                    for (int nt = 0; nt < L.n_tiles && ok; ++nt, ++lt) {
                        const int acc = lt & 1;
                        const uint32_t acc_phase = (lt >> 1) & 1;
                        if (!mbar_wait(&bars->acc_empty[acc], acc_phase ^ 1) || *abort_flag) { ok = false; break; }
                        tcgen05_fence_after();
                        const uint32_t d = tmem_base + (uint32_t)(acc * kAccCols);
                        // pass 1: cross terms
                        for (int kb = 0; kb < num_kb; ++kb) {
                            if (nt == 0) {
                                // block kb of the panel is complete
                                if (!mbar_wait_cluster(&bars->a_ready[kb], (a_phase >> kb) & 1u) || *abort_flag) { ok = false; break; }
                                a_phase ^= 1u << kb;
                            }
                            if (!mbar_wait(&bars->full[s], phase) || *abort_flag) { ok = false; break; }
                            tcgen05_fence_after();
                            const uint32_t st = smem_u32(Bst + (size_t)s * kStageBytes);
                            const uint64_t da_hi = make_desc(a_hi0 + (uint32_t)kb * kABlockBytes);
                            const uint64_t da_lo = make_desc(a_lo0 + (uint32_t)kb * kABlockBytes);
                            const uint64_t db_hi = make_desc(st);
                            const uint64_t db_lo = make_desc(st + kBChunkBytes);
#pragma unroll
                            for (int k = 0; k < BKH / 16; ++k) {
                                if (kb * (BKH / 16) + k >= ksteps) break;
                                const uint64_t ko = (uint64_t)(k * 2);   // 16 halves = 32 bytes = 2 x 16-byte units
                                mma_f16<CTAS>(d, da_lo + ko, db_hi + ko, idesc, (kb | k) ? 1u : 0u);
                                mma_f16<CTAS>(d, da_hi + ko, db_lo + ko, idesc, 1u);
                                if (ONEPASS) mma_f16<CTAS>(d, da_hi + ko, db_hi + ko, idesc, 1u);
                            }
                            tcgen05_commit<CTAS>(&bars->empty[s]);
                            if (++s == stages) { s = 0; phase ^= 1; }
                        }
                        // pass 2: hi * hi on top of the cross terms scaled by 2^-11
                        for (int kb = 0; !ONEPASS && kb < num_kb && ok; kb += 2) {
                            if (!mbar_wait(&bars->full[s], phase) || *abort_flag) { ok = false; break; }
                            tcgen05_fence_after();
                            const uint32_t st = smem_u32(Bst + (size_t)s * kStageBytes);
                            const int blocks = kb + 1 < num_kb ? 2 : 1;
                            for (int h = 0; h < blocks; ++h) {
                                const uint64_t da = make_desc(a_hi0 + (uint32_t)(kb + h) * kABlockBytes);
                                const uint64_t db = make_desc(st + (uint32_t)h * kBChunkBytes);
#pragma unroll
                                for (int k = 0; k < BKH / 16; ++k) {
                                    if ((kb + h) * (BKH / 16) + k >= ksteps) break;
                                    const uint64_t ko = (uint64_t)(k * 2);
                                    if (kb == 0 && h == 0 && k == 0) mma_f16_pair_scaled<11>(d, da + ko, db + ko, idesc);
                                    else mma_f16<CTAS>(d, da + ko, db + ko, idesc, 1u);
                                }
                            }
                            tcgen05_commit<CTAS>(&bars->empty[s]);
                            if (++s == stages) { s = 0; phase ^= 1; }
                        }
                        if (ok) tcgen05_commit<CTAS>(&bars->acc_full[acc]);
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicOr(a.status, 1);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (8 warps)
        const int ew = warp - 2;
        const int quarter = warp & 3;                       // TMEM lane quarter this warp may read
        const int col_group = ew >> 2;                        // which of the quarter's warps: it takes every kChainColGroups-th 32-column chunk
        const int prow = quarter * 32 + lane;               // this thread's row of the CTA's panel
        const uint32_t a_hi0 = smem_u32(A_hi), a_lo0 = smem_u32(A_lo);
        const uint32_t acc_empty_addr0 = map_to_cta(smem_u32(&bars->acc_empty[0]), 0);
        const uint32_t a_ready_addr = map_to_cta(smem_u32(&bars->a_ready[0]), 0);
        bool ok = true, out_of_range = false;
        int lt = 0, vstep = 0;
        // one-pass form: the coefficients and the row constant are held times q_scale throughout (every factor is a
        // power of two, so the results are those of the unscaled arithmetic); the constant is scaled back as it leaves
        const float q_scale = ONEPASS ? a.q_scale : 1.0f;
        constexpr float lo_scale = ONEPASS ? 1.0f : kLoScale;
        for (long long p = group; p < n_panels && ok; p += n_groups) {
            const long long r = p * (BM * CTAS) + (long long)rank * BM + prow;
            const bool row_ok = r < a.M;
            const long long rr = row_ok ? r : 0;
            const int b = (int)(rr / (2LL * a.n_k));
            const int upper = (int)((rr / a.n_k) & 1);
            const int i = (int)(rr % a.n_k);
            float dacc = (col_group == 0) ? a.bias_k[i] * q_scale : 0.0f;
            {
                // start: row i of W_k through the ReLU of layer k-1; the constant takes the nu terms and Q.b
                const ChainLayer &Lk = P.layer[a.k];
                const int n = Lk.n_in;
                const int kp = (n + BKH - 1) / BKH * BKH;
                const size_t relax_row = (size_t)b * Lk.ld_in;
                const float *wrow = a.Wk + (size_t)i * a.ldw_k;
                for (int c0 = 32 * col_group; c0 < kp; c0 += 32 * kChainColGroups) {
                    float q[32];
                    if (c0 < Lk.ld_in && row_ok) {
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const int col = c0 + g * 4;
                            const float4 w4 = *reinterpret_cast<const float4 *>(wrow + col);
                            const float4 bz = *reinterpret_cast<const float4 *>(Lk.bias_below + col);
                            const float c4[4] = {w4.x, w4.y, w4.z, w4.w}, b4[4] = {bz.x, bz.y, bz.z, bz.w};
                            float l4[4] = {1.0f, 1.0f, 1.0f, 1.0f}, u4[4] = {1.0f, 1.0f, 1.0f, 1.0f},
                                  n4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                            if (Lk.relu_below) {
                                const float4 ll = *reinterpret_cast<const float4 *>(Lk.lamL + relax_row + col);
                                const float4 lu = *reinterpret_cast<const float4 *>(Lk.lamU + relax_row + col);
                                const float4 nu = *reinterpret_cast<const float4 *>(Lk.nuU + relax_row + col);
                                l4[0] = ll.x; l4[1] = ll.y; l4[2] = ll.z; l4[3] = ll.w;
                                u4[0] = lu.x; u4[1] = lu.y; u4[2] = lu.z; u4[3] = lu.w;
                                n4[0] = nu.x; n4[1] = nu.y; n4[2] = nu.z; n4[3] = nu.w;
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float x = 0.0f;
                                if (col + e < n) {
                                    const float c = c4[e] * q_scale;
                                    const bool nonneg = (c >= 0.0f);
                                    const bool use_lower = upper ? !nonneg : nonneg;
                                    x = c * (use_lower ? l4[e] : u4[e]);
                                    dacc = fmaf(c, use_lower ? 0.0f : n4[e], dacc);
                                    dacc = fmaf(x, b4[e], dacc);
                                }
                                q[g * 4 + e] = x;
                            }
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) q[e] = 0.0f;
                    }
                    write_panel_chunk(a_hi0, a_lo0, prow, c0, q, row_ok, out_of_range, lo_scale);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(a_ready_addr + (uint32_t)((c0 >> 6) * sizeof(uint64_t)));
                }
            }
            // boxes of this CTA's 128 rows (the producer stages the vectors of the first two)
            const long long cta_row0 = p * (BM * CTAS) + (long long)rank * BM;
            const long long cta_last = (cta_row0 + BM - 1 < a.M ? cta_row0 + BM - 1 : a.M - 1);
            const int b_last = (int)(cta_last / (2LL * a.n_k));
            int b_first = (int)(cta_row0 / (2LL * a.n_k));
            if (b_first > b_last) b_first = b_last;
            const int nb = b_last - b_first + 1 < 2 ? b_last - b_first + 1 : 2;
            for (int j = a.k - 1; j >= a.j_end && ok; --j) {
                const ChainLayer &L = P.layer[j];
                const bool last = (j == a.j_end);
                const size_t relax_row = (size_t)b * L.ld_in;
                // the step's descriptor in registers (the table is indexed by j)
                const int ld_in = L.ld_in, n_in = L.n_in, bn = L.bn, n_tiles = L.n_tiles, relu_below = L.relu_below;
                const float *lamL = L.lamL + relax_row, *lamU = L.lamU + relax_row, *nuU = L.nuU + relax_row;
                const float *bias_below = L.bias_below;
                const float acc_scale = ONEPASS ? L.w_unscale : 1.0f;     // the accumulator holds 2^s times the product
                // staged copies of these vectors (the producer fetched them while the MMAs ran): the bias always,
                // the relaxation for rows of the CTA's first two boxes
                const int vbuf = (a.vec_ld > 0 && !last) ? (vstep & 1) : -1;
                if (vbuf >= 0) {
                    const float *vs = vec_stage + (size_t)vbuf * vec_floats;
                    bias_below = vs;
                    const int sb = b - b_first;
                    if (sb >= 0 && sb < nb) {
                        lamL = vs + a.vec_ld + (size_t)sb * 3 * a.vec_ld;
                        lamU = lamL + a.vec_ld;
                        nuU = lamU + a.vec_ld;
                    }
                }
                for (int nt = 0; nt < n_tiles && ok; ++nt, ++lt) {
                    const int acc = lt & 1;
                    const uint32_t acc_phase = (lt >> 1) & 1;
                    if (!mbar_wait(&bars->acc_full[acc], acc_phase) || *abort_flag) { ok = false; break; }
                    if (vbuf >= 0 && (!mbar_wait(&bars->vec_full[vbuf], (vstep >> 1) & 1) || *abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kAccCols);
                    if (!last) {
                        // ReLU back-step through the neurons below layer j; the result is the next step's operand.
                        // (A step that is not the last has a single column tile: n_in <= 256.)
                        const int kp = (n_in + BKH - 1) / BKH * BKH;
                        for (int c0 = 32 * col_group; c0 < kp; c0 += 32 * kChainColGroups) {
                            float q[32];
                            if (c0 < ld_in) {
                                uint32_t v[32];
                                __syncwarp();
                                tmem_ld32(t_addr + (uint32_t)c0, v);
                                tmem_ld_wait();
#pragma unroll
                                for (int g = 0; g < 8; ++g) {
                                    const int col = c0 + g * 4;
                                    const float4 bz = *reinterpret_cast<const float4 *>(bias_below + col);
                                    const float b4[4] = {bz.x, bz.y, bz.z, bz.w};
                                    if (relu_below) {
                                        const float4 ll = *reinterpret_cast<const float4 *>(lamL + col);
                                        const float4 lu = *reinterpret_cast<const float4 *>(lamU + col);
                                        const float4 nu = *reinterpret_cast<const float4 *>(nuU + col);
                                        const float l4[4] = {ll.x, ll.y, ll.z, ll.w}, u4[4] = {lu.x, lu.y, lu.z, lu.w},
                                                    n4[4] = {nu.x, nu.y, nu.z, nu.w};
#pragma unroll
                                        for (int e = 0; e < 4; ++e) {
                                            const float c = __uint_as_float(v[g * 4 + e]) * acc_scale;
                                            const bool nonneg = (c >= 0.0f);
                                            const bool use_lower = upper ? !nonneg : nonneg;
                                            q[g * 4 + e] = c * (use_lower ? l4[e] : u4[e]);
                                            dacc = fmaf(c, use_lower ? 0.0f : n4[e], dacc);
                                        }
                                    } else {
#pragma unroll
                                        for (int e = 0; e < 4; ++e) q[g * 4 + e] = __uint_as_float(v[g * 4 + e]) * acc_scale;
                                    }
#pragma unroll
                                    for (int e = 0; e < 4; ++e) dacc = fmaf(q[g * 4 + e], b4[e], dacc);
                                }
                            } else {
#pragma unroll
                                for (int e = 0; e < 32; ++e) q[e] = 0.0f;
                            }
                            write_panel_chunk(a_hi0, a_lo0, prow, c0, q, row_ok, out_of_range, lo_scale);
                            fence_async_smem();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(a_ready_addr + (uint32_t)((c0 >> 6) * sizeof(uint64_t)));
                        }
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive_cluster(acc_empty_addr0 + (uint32_t)(acc * sizeof(uint64_t)));
                            if (vbuf >= 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->vec_empty[vbuf]), rank));
                        }
                    } else {
                        // map(simplify_lower/upper) against the concrete bounds of what the traversal reached
                        for (int c0 = 32 * col_group; c0 < bn; c0 += 32 * kChainColGroups) {
                            const int col0 = nt * bn + c0;
                            if (col0 >= ld_in) break;              // warp-uniform; ld_in is a multiple of 32
                            uint32_t v[32];
                            __syncwarp();
                            tmem_ld32(t_addr + (uint32_t)c0, v);
                            tmem_ld_wait();
                            const float *lrow = a.box_l + relax_row + col0;
                            const float *urow = a.box_u + relax_row + col0;
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                const float4 l4 = *reinterpret_cast<const float4 *>(lrow + g * 4);
                                const float4 u4 = *reinterpret_cast<const float4 *>(urow + g * 4);
                                const float lo4[4] = {l4.x, l4.y, l4.z, l4.w}, up4[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float c = __uint_as_float(v[g * 4 + e]) * acc_scale;
                                    const bool nonneg = (c >= 0.0f);
                                    dacc = fmaf(c, (nonneg != (upper != 0)) ? lo4[e] : up4[e], dacc);
                                }
                            }
                        }
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acc_empty_addr0 + (uint32_t)(acc * sizeof(uint64_t)));
                    }
                }
                if (vbuf >= 0) ++vstep;
            }
            if (ok && row_ok) CERT_ST(a.d_out[(size_t)col_group * a.slot_stride + r], ONEPASS ? dacc * a.q_unscale : dacc);
        }
        if (out_of_range) atomicOr(a.status, 2);
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(a.status, 1);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();      // no CTA leaves while its peer may still reach into it
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)(2 * kAccCols))
                     : "memory");
    }
}

}  // namespace

int chain16_smem_bytes(int a_blocks, int max_bnl, int ld_max, int *stages, int *b_chunk_bytes, int *vec_ld) {
    const int chunk = (max_bnl * BKH * 2 + 1023) / 1024 * 1024;
    const int stage = 2 * chunk;
    const int fixed = 2 * a_blocks * kABlockBytes + (int)sizeof(BarriersChain) + 1024;
    const int vec_bytes = 2 * 7 * ld_max * (int)sizeof(float);
    *b_chunk_bytes = chunk;
    // the staging buffers are taken if three pipeline stages still fit beside them
    int st = (kTcSmemMax - fixed - vec_bytes) / stage;
    *vec_ld = ld_max;
    if (st < 3) {
        st = (kTcSmemMax - fixed) / stage;
        *vec_ld = 0;
    }
    if (st > 8) st = 8;
    *stages = st;
    return fixed + (*vec_ld ? vec_bytes : 0) + (st > 0 ? st : 0) * stage;
}

bool chain16_prepare() {
    if (cudaFuncSetAttribute(chain16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax) != cudaSuccess ||
        cudaFuncSetAttribute(chain16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

void launch_chain16(const ChainParams &P, const ChainArgs &a, int pairs, int smem_bytes, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(pairs * CTAS), 1, 1);
    cfg.blockDim = dim3(kThreadsChain, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CTAS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    if (a.one_pass) cudaLaunchKernelEx(&cfg, chain16_kernel<true>, P, a);
    else cudaLaunchKernelEx(&cfg, chain16_kernel<false>, P, a);
}

}  // namespace cert
