// Affine back-step on the tensor cores with an fp16 split (three fp16 products per fp32-accurate
// multiply-add), the ReLU back-step or the concretisation fused into the epilogue.
//
//   P = Q * W_j   (Section 4.3, Matmul rewrite of the traversal step), then as in gemm_tc.cu.
//
// x = hi + 2^-11 * lo with hi = fp16(x), lo = fp16(2^11 * (x - hi)).  A tile takes two passes over K into
// one fp32 accumulator in tensor memory:
//   pass 1:  D  = sum over K of  Q_lo * W_hi + Q_hi * W_lo      (cross terms, in units of 2^-11)
//   pass 2:  D  = Q_hi * W_hi + D * 2^-11  for the first k-step (the MMA scales its input accumulator),
//            D += Q_hi * W_hi             for the rest.
// fp16 products are exact in fp32, so the result has the accuracy of the 3xTF32 form at twice the MMA rate;
// pass 2 stages only the hi tiles (two k-blocks per pipeline stage).  A coefficient beyond the fp16 range
// raises bit 1 of the status word.
//
// ONEPASS: both operands carry a power of two, Q' = 2^a Q and W' = 2^s W (a per traversal, s per layer), large
// enough that the lo parts need no factor of their own to stay normal fp16 numbers: x' = hi + lo with
// hi = fp16(x'), lo = fp16(x' - hi).  The three products then share one scale,
//   D += Q_lo * W_hi + Q_hi * W_lo + Q_hi * W_hi,
// so a k-block is staged once (four tiles) for all of them and the epilogue multiplies by 2^-(a+s).  The two-pass
// form stages six tiles per k-block.  The kernel is bound by what an SM takes in from L2 per cycle (a plain
// fp16 GEMM of this tile shape needs the same 64 bytes per cycle and SM as the two-pass form), so fewer staged
// bytes per product are what raises the tensor pipe's share.  The price is range: |Q| 2^a must stay in the fp16
// range, where the two-pass form only needs |Q| to.
//
// CTA pairs (tcgen05 cta_group::2) on 256-row panels, persistent over (row panel, column tile) work tiles,
// two accumulators so that the epilogue of a tile overlaps the MMAs of the next, as in gemm_tc.cu.  A tile's
// MMAs take half the time they take there, so eight epilogue warps (two per TMEM lane quarter, taking
// alternate 32-column chunks) run the epilogue.  A row's constant for this tile is written by both of its
// owner threads: 2 * n_tiles slots per row, summed in slot order by the next kernel.
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "gemm_tc16.cuh"
#include "tc_ptx.cuh"

namespace cert {

namespace {

constexpr int BM = 128;                  // rows per CTA
constexpr int BKH = 64;                  // halves of K per stage: one 128-byte swizzle row
constexpr int kEpiWarps = 8;
constexpr int kThreads16 = 64 + kEpiWarps * 32;
constexpr int kATileBytes = BM * BKH * 2;
constexpr int kSlabBytes16 = 32 * 64;    // 32 rows x 32 halves per epilogue warp and output array
constexpr int kEpiBytes16 = kEpiWarps * 2 * kSlabBytes16;

struct __align__(8) Barriers16 {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int EPI, bool ONEPASS>
__global__ void __launch_bounds__(kThreads16, 1)
gemm_tc16_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                 const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                 const __grid_constant__ CUtensorMap map_o_hi, const __grid_constant__ CUtensorMap map_o_lo,
                 const TcArgs a) {
    constexpr int CTAS = 2;
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.bn;
    const int BNL = BN / CTAS;                 // rows of the W_j tile this CTA stages
    const int stages = a.stages;
    const uint32_t b_tile_bytes = (uint32_t)BNL * BKH * 2;
    const uint32_t stage_bytes = 2 * kATileBytes + 2 * b_tile_bytes;
    uint8_t *epi_smem = smem + (size_t)stages * stage_bytes;
    Barriers16 *bars = reinterpret_cast<Barriers16 *>(epi_smem + kEpiBytes16);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (a.K + BKH - 1) / BKH;
    const int n_tiles = a.n_tiles;
    const int total_tiles = a.total_tiles;
    const uint32_t rank = cluster_ctarank();
    const int group = (int)cluster_id_x();
    const int n_groups = (int)num_clusters_x();

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->acc_full[i], 1);
            mbar_init(&bars->acc_empty[i], kEpiWarps * CTAS);
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&bars->tmem_base)),
                     "r"((uint32_t)a.tmem_cols)
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
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            int armed = 0;
            for (int t = group; t < total_tiles && ok; t += n_groups) {
                const int row0 = (t / n_tiles) * (BM * CTAS) + (int)rank * BM;
                // the last n_narrow column tiles are 32 columns narrower: this CTA's half of W_j's rows starts
                // accordingly (the TMA box keeps its size; the rows beyond the half are not read by the MMAs)
                const int nt = t % n_tiles;
                const int narrow = nt - (n_tiles - a.n_narrow);
                const int col0 = nt * BN - (narrow > 0 ? narrow * 32 : 0) + (int)rank * (narrow >= 0 ? BNL - 16 : BNL);
                // pass 1: all four tiles of a k-block per stage
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (!mbar_wait(&bars->empty[s], phase ^ 1) || *abort_flag) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * stage_bytes;
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[s], stage_bytes * CTAS);
                    const uint32_t bar = map_to_cta(smem_u32(&bars->full[s]), 0);
                    const int kx = kb * BKH;
                    tma_load_2d<CTAS>(smem_u32(st), &map_a_hi, bar, kx, row0);
                    tma_load_2d<CTAS>(smem_u32(st + kATileBytes), &map_a_lo, bar, kx, row0);
                    tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes), &map_b_hi, bar, kx, col0);
                    tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes + b_tile_bytes), &map_b_lo, bar, kx, col0);
                    ++armed;
                    if (++s == stages) { s = 0; phase ^= 1; }
                }
                // pass 2: the hi tiles of two k-blocks per stage (the second in the slots of the lo tiles)
                for (int kb = 0; !ONEPASS && kb < num_kb && ok; kb += 2) {
                    if (!mbar_wait(&bars->empty[s], phase ^ 1) || *abort_flag) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * stage_bytes;
                    const bool two = kb + 1 < num_kb;
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[s], (two ? stage_bytes : stage_bytes / 2) * CTAS);
                    const uint32_t bar = map_to_cta(smem_u32(&bars->full[s]), 0);
                    tma_load_2d<CTAS>(smem_u32(st), &map_a_hi, bar, kb * BKH, row0);
                    tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes), &map_b_hi, bar, kb * BKH, col0);
                    if (two) {
                        tma_load_2d<CTAS>(smem_u32(st + kATileBytes), &map_a_hi, bar, (kb + 1) * BKH, row0);
                        tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes + b_tile_bytes), &map_b_hi, bar, (kb + 1) * BKH, col0);
                    }
                    ++armed;
                    if (++s == stages) { s = 0; phase ^= 1; }
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
            // kind::f16: D = f32, A = B = f16 (format 0), both K-major
            const uint32_t idesc_wide = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CTAS) >> 4) << 24);
            const uint32_t idesc_narrow = (1u << 4) | ((uint32_t)((BN - 32) >> 3) << 17) | ((uint32_t)((BM * CTAS) >> 4) << 24);
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            int lt = 0;
            for (int t = group; t < total_tiles && ok; t += n_groups, ++lt) {
                const int acc = lt & 1;
                const uint32_t acc_phase = (lt >> 1) & 1;
                if (!mbar_wait(&bars->acc_empty[acc], acc_phase ^ 1) || *abort_flag) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d = tmem_base + (uint32_t)(acc * BN);
                const uint32_t idesc = (t % n_tiles) >= n_tiles - a.n_narrow ? idesc_narrow : idesc_wide;
                // pass 1: cross terms
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (!mbar_wait(&bars->full[s], phase) || *abort_flag) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t st = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t da_hi = make_desc(st);
                    const uint64_t da_lo = make_desc(st + kATileBytes);
                    const uint64_t db_hi = make_desc(st + 2 * kATileBytes);
                    const uint64_t db_lo = make_desc(st + 2 * kATileBytes + b_tile_bytes);
#pragma unroll
                    for (int k = 0; k < BKH / 16; ++k) {
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
                    const uint32_t st = smem_u32(smem + (size_t)s * stage_bytes);
                    const int blocks = kb + 1 < num_kb ? 2 : 1;
                    for (int h = 0; h < blocks; ++h) {
                        const uint64_t da = make_desc(st + (uint32_t)h * kATileBytes);
                        const uint64_t db = make_desc(st + 2 * kATileBytes + (uint32_t)h * b_tile_bytes);
#pragma unroll
                        for (int k = 0; k < BKH / 16; ++k) {
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
            if (!ok) {
                *abort_flag = 1;
                atomicOr(a.status, 1);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (8 warps)
        const int ew = warp - 2;
        const int quarter = warp & 3;                       // TMEM lane quarter this warp may read
        const int half_id = ew >> 2;                        // which of the two warps of the quarter
        uint8_t *slab_hi = epi_smem + (size_t)ew * 2 * kSlabBytes16;
        uint8_t *slab_lo = slab_hi + kSlabBytes16;
        const uint32_t acc_empty_addr0 = map_to_cta(smem_u32(&bars->acc_empty[0]), 0);
        bool ok = true, out_of_range = false;
        int lt = 0;
        for (int t = group; t < total_tiles && ok; t += n_groups, ++lt) {
            const int nt = t % n_tiles;
            const long long warp_row0 = (long long)(t / n_tiles) * (BM * CTAS) + (int)rank * BM + quarter * 32;
            const long long r = warp_row0 + lane;
            const bool row_ok = r < a.M;
            const long long rr = row_ok ? r : 0;
            const int b = (int)(rr / (2LL * a.n_k));
            const int upper = (int)((rr / a.n_k) & 1);
            const size_t relax_row = (size_t)b * a.ld_n;
            float dacc = 0.0f;
            const int acc = lt & 1;
            const uint32_t acc_phase = (lt >> 1) & 1;
            if (!mbar_wait(&bars->acc_full[acc], acc_phase) || *abort_flag) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
            const int narrow = nt - (n_tiles - a.n_narrow);
            const int tile_col0 = nt * BN - (narrow > 0 ? narrow * 32 : 0);
            const int tile_cols = narrow >= 0 ? BN - 32 : BN;
            for (int c0 = 32 * half_id; c0 < tile_cols; c0 += 64) {
                const int col0 = tile_col0 + c0;
                if (col0 >= a.ld_n) break;                   // warp-uniform; ld_n is a multiple of 32
                uint32_t v[32];
                // a residual connection ends on these neurons: its waiting coefficients (an fp16 pair here) for the
                // warp's 32 rows x 32 columns are requested before the accumulator is read, eight rows (64-byte
                // pieces of a row) per instruction: load i brings 16-byte piece lane % 4 of row 8 i + lane / 4
                uint4 ch[EPI == TC_EPI_RELU_SKIP ? 4 : 1], cl[EPI == TC_EPI_RELU_SKIP ? 4 : 1];
                const bool joins = EPI == TC_EPI_RELU_SKIP && a.add_hi != nullptr;
                if (EPI == TC_EPI_RELU_SKIP && joins) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        long long rw = warp_row0 + 8 * i + (lane >> 2);
                        if (rw >= a.M) rw = 0;
                        const size_t o = (size_t)rw * a.ld_n + col0 + (lane & 3) * 8;
                        ch[i] = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(a.add_hi) + o));
                        cl[i] = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(a.add_lo) + o));
                    }
                }
                __syncwarp();
                tmem_ld32(t_addr + (uint32_t)c0, v);
                tmem_ld_wait();
                if (ONEPASS) {
                    // the accumulator holds 2^(a+s) times the product
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * a.acc_scale);
                }
                if (EPI == TC_EPI_RELU || EPI == TC_EPI_RELU_SKIP) {
                    // the slab is free again once the previous chunk's stores have read it
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                    const uint32_t row_hi = smem_u32(slab_hi) + (uint32_t)lane * 64u;
                    const uint32_t row_lo = smem_u32(slab_lo) + (uint32_t)lane * 64u;
                    if (EPI == TC_EPI_RELU_SKIP && joins) {
                        // through the (free) slab to the lane that owns the row; a lane then reads and rewrites
                        // only its own row
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t rw = (uint32_t)(8 * i + (lane >> 2));
                            const uint32_t off = rw * 64u + ((((uint32_t)lane & 3u) ^ ((rw >> 1) & 3u)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(slab_hi) + off),
                                         "r"(ch[i].x), "r"(ch[i].y), "r"(ch[i].z), "r"(ch[i].w) : "memory");
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(slab_lo) + off),
                                         "r"(cl[i].x), "r"(cl[i].y), "r"(cl[i].z), "r"(cl[i].w) : "memory");
                        }
                        __syncwarp();
                    }
#pragma unroll
                    for (int c16 = 0; c16 < 4; ++c16) {
                        uint32_t ph[4], pl[4];              // 8 halves of hi, 8 of lo
                        uint32_t jh[4] = {0u, 0u, 0u, 0u}, jl[4] = {0u, 0u, 0u, 0u};     // the joining pair's 8 columns
                        if (EPI == TC_EPI_RELU_SKIP && joins) {
                            const uint32_t swj = (uint32_t)((c16 ^ ((lane >> 1) & 3)) << 4);
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(jh[0]), "=r"(jh[1]), "=r"(jh[2]),
                                         "=r"(jh[3]) : "r"(row_hi + swj) : "memory");
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(jl[0]), "=r"(jl[1]), "=r"(jl[2]),
                                         "=r"(jl[3]) : "r"(row_lo + swj) : "memory");
                        }
#pragma unroll
                        for (int g2 = 0; g2 < 2; ++g2) {
                            const int g = c16 * 2 + g2;
                            const int col = col0 + g * 4;
                            float q[4];
                            const float4 bz = *reinterpret_cast<const float4 *>(a.bias_below + col);
                            if (EPI == TC_EPI_RELU_SKIP) {
                                // the waiting coefficients and the unit coefficient join before the ReLU back-step
                                float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                                if (joins) {
                                    const uint2 sh = make_uint2(jh[g2 * 2], jh[g2 * 2 + 1]);
                                    const uint2 sl = make_uint2(jl[g2 * 2], jl[g2 * 2 + 1]);
                                    const __half2 h01 = *reinterpret_cast<const __half2 *>(&sh.x), h23 = *reinterpret_cast<const __half2 *>(&sh.y);
                                    const __half2 l01 = *reinterpret_cast<const __half2 *>(&sl.x), l23 = *reinterpret_cast<const __half2 *>(&sl.y);
                                    const float2 fh01 = __half22float2(h01), fh23 = __half22float2(h23);
                                    const float2 fl01 = __half22float2(l01), fl23 = __half22float2(l23);
                                    if (ONEPASS) {
                                        // a pair of this traversal: 2^a times the coefficient, lo unscaled
                                        s4[0] = (fh01.x + fl01.x) * a.q_unscale; s4[1] = (fh01.y + fl01.y) * a.q_unscale;
                                        s4[2] = (fh23.x + fl23.x) * a.q_unscale; s4[3] = (fh23.y + fl23.y) * a.q_unscale;
                                    } else {
                                        const float inv = 1.0f / kLoScale;
                                        s4[0] = fmaf(fl01.x, inv, fh01.x); s4[1] = fmaf(fl01.y, inv, fh01.y);
                                        s4[2] = fmaf(fl23.x, inv, fh23.x); s4[3] = fmaf(fl23.y, inv, fh23.y);
                                    }
                                }
                                const int own = a.add_identity ? (int)(rr % a.n_k) : -1;
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    v[g * 4 + e] = __float_as_uint(__uint_as_float(v[g * 4 + e]) + s4[e] +
                                                                   (col + e == own ? 1.0f : 0.0f));
                            }
                            if (a.has_relu) {
                                const float4 ll = *reinterpret_cast<const float4 *>(a.lamL + relax_row + col);
                                const float4 lu = *reinterpret_cast<const float4 *>(a.lamU + relax_row + col);
                                const float4 nu = *reinterpret_cast<const float4 *>(a.nuU + relax_row + col);
                                const float l4[4] = {ll.x, ll.y, ll.z, ll.w}, u4[4] = {lu.x, lu.y, lu.z, lu.w},
                                            n4[4] = {nu.x, nu.y, nu.z, nu.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float c = __uint_as_float(v[g * 4 + e]);
                                    const bool nonneg = (c >= 0.0f);
                                    const bool use_lower = upper ? !nonneg : nonneg;
                                    q[e] = c * (use_lower ? l4[e] : u4[e]);
                                    dacc = fmaf(c, use_lower ? 0.0f : n4[e], dacc);
                                }
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    q[e] = __uint_as_float(v[g * 4 + e]);
                            }
                            dacc = fmaf(q[0], bz.x, dacc);
                            dacc = fmaf(q[1], bz.y, dacc);
                            dacc = fmaf(q[2], bz.z, dacc);
                            dacc = fmaf(q[3], bz.w, dacc);
                            __half h[4], l[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float x = ONEPASS ? q[e] * a.q_scale : q[e];
                                out_of_range |= row_ok && !(fabsf(x) <= 60000.0f);
                                h[e] = __float2half_rn(x);
                                l[e] = __float2half_rn(ONEPASS ? x - __half2float(h[e]) : (x - __half2float(h[e])) * kLoScale);
                            }
                            ph[g2 * 2 + 0] = (uint32_t)__half_as_ushort(h[0]) | ((uint32_t)__half_as_ushort(h[1]) << 16);
                            ph[g2 * 2 + 1] = (uint32_t)__half_as_ushort(h[2]) | ((uint32_t)__half_as_ushort(h[3]) << 16);
                            pl[g2 * 2 + 0] = (uint32_t)__half_as_ushort(l[0]) | ((uint32_t)__half_as_ushort(l[1]) << 16);
                            pl[g2 * 2 + 1] = (uint32_t)__half_as_ushort(l[2]) | ((uint32_t)__half_as_ushort(l[3]) << 16);
                        }
                        // 16-byte chunk c16 of this lane's 64-byte slab row, at its 64-byte-swizzle position
                        const uint32_t sw = (uint32_t)((c16 ^ ((lane >> 1) & 3)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_hi + sw), "r"(ph[0]), "r"(ph[1]),
                                     "r"(ph[2]), "r"(ph[3]) : "memory");
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_lo + sw), "r"(pl[0]), "r"(pl[1]),
                                     "r"(pl[2]), "r"(pl[3]) : "memory");
                    }
                    fence_async_smem();
                    __syncwarp();
                    // rows past the end of the matrix land in scratch rows of the workspace or are clipped
                    if (lane == 0) {
                        tma_store_2d(&map_o_hi, smem_u32(slab_hi), col0, (int)warp_row0);
                        tma_store_2d(&map_o_lo, smem_u32(slab_lo), col0, (int)warp_row0);
                        tma_store_commit();
                    }
                } else if (EPI == TC_EPI_REUSE) {
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                    const int bx = (int)(rr / a.reuse_R), s_in = (int)(rr % a.reuse_R);
                    const bool is_const = s_in == a.reuse_n0;
                    const bool is_coord = s_in < a.reuse_n0;
                    const float lo_s = is_coord ? a.l0[(size_t)bx * a.reuse_ld0 + s_in] : 0.0f;
                    const float up_s = is_coord ? a.u0[(size_t)bx * a.reuse_ld0 + s_in] : 0.0f;
                    const uint32_t row_hi = smem_u32(slab_hi) + (uint32_t)lane * 128u;   // the warp's two fp16 slabs as one fp32 slab
                    float w[32];
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        float q[4];
                        const float4 bz = *reinterpret_cast<const float4 *>(a.bias2 + col0 + g * 4);
                        const float b4[4] = {bz.x, bz.y, bz.z, bz.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int col = col0 + g * 4 + e;
                            float c = __uint_as_float(v[g * 4 + e]);
                            if (is_const) c += b4[e];
                            q[e] = c;
                            // simplify_lower for a lower shape, simplify_upper for an upper one; the constant as it is
                            const bool upper_col = col >= a.n_half;
                            const bool nonneg = (c >= 0.0f);
                            float term = c * ((nonneg != upper_col) ? lo_s : up_s);
                            if (is_const) term = c;
                            w[g * 4 + e] = (row_ok && col < 2 * a.n_half) ? term : 0.0f;
                        }
                        const uint32_t sw = (uint32_t)((g ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(row_hi + sw), "f"(q[0]),
                                     "f"(q[1]), "f"(q[2]), "f"(q[3]) : "memory");
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&map_o_hi, smem_u32(slab_hi), col0, (int)warp_row0);
                        tma_store_commit();
                    }
                    // Column sums over the warp's 32 rows by recursive halving: after the step with
                    // distance d a lane keeps the columns whose index has the lane's bit d, so lane L
                    // ends with column L.  Fixed order.
#pragma unroll
                    for (int d = 16; d >= 1; d >>= 1) {
                        const bool hi_half = (lane & d) != 0;
#pragma unroll
                        for (int j = 0; j < d; ++j) {
                            const float send = hi_half ? w[j] : w[j + d];
                            const float keep = hi_half ? w[j + d] : w[j];
                            w[j] = keep + __shfl_xor_sync(0xffffffffu, send, d);
                        }
                    }
                    if (warp_row0 < a.M) CERT_ST(a.colsum[(size_t)(warp_row0 >> 5) * a.ld_n + col0 + lane], w[0]);
                } else if (row_ok) {
                    const float *lrow = a.l0 + (size_t)b * a.ld_n + col0;
                    const float *urow = a.u0 + (size_t)b * a.ld_n + col0;
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const float4 l4 = *reinterpret_cast<const float4 *>(lrow + g * 4);
                        const float4 u4 = *reinterpret_cast<const float4 *>(urow + g * 4);
                        const float lo4[4] = {l4.x, l4.y, l4.z, l4.w}, up4[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float c = __uint_as_float(v[g * 4 + e]);
                            const bool nonneg = (c >= 0.0f);
                            dacc = fmaf(c, (nonneg != (upper != 0)) ? lo4[e] : up4[e], dacc);
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_addr0 + (uint32_t)(acc * sizeof(uint64_t)));
            // This warp's share of the row constant (of the bound) goes to slot 2*nt + half_id; the first
            // slot also carries the constant so far.
            if (EPI != TC_EPI_REUSE && row_ok) {
                float tot = dacc;
                if (nt == 0 && half_id == 0) {
                    float prev = 0.0f;
                    for (int sidx = 0; sidx < a.n_slots_in; ++sidx) prev += a.d_in[(size_t)sidx * a.slot_stride + r];
                    tot += prev;
                }
                CERT_ST(a.d_out[(size_t)(2 * nt + half_id) * a.slot_stride + r], tot);
            }
        }
        if (EPI != TC_EPI_CONCRETIZE && lane == 0) tma_store_wait_all();
        if (__any_sync(0xffffffffu, out_of_range) && lane == 0) atomicOr(a.status, 2);
        if (!ok && lane == 0) atomicOr(a.status, 1);
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();      // no CTA leaves while its peer may still reach into it
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols)
                     : "memory");
    }
}

__device__ __forceinline__ float warp_sum16(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Start of a back-substitution at FC layer k as an fp16 pair: row i of W_k pushed through the ReLU below,
// constant = b_k[i] + the nu terms + Q.b of the layer below.  The pair is hi = fp16(q_scale x),
// lo = fp16(lo_scale (q_scale x - hi)): (1, 2^11) for the two-pass contraction, (2^a, 1) for the one-pass one.
// A warp takes kRowsPerWarp consecutive neurons of one (box, side), 8 columns per lane: the relaxation and bias
// vectors are read once for those rows.
constexpr int kRowsPerWarp = 4;

// three 256-thread blocks per SM: the kernel only writes, and needs the warps in flight
__global__ void __launch_bounds__(256, 3)
expr_start16_kernel(const float *__restrict__ Wk, int ldw_k, const float *__restrict__ bias_k, __half *__restrict__ Q_hi,
                    __half *__restrict__ Q_lo, float *__restrict__ d, long long n_warps, int n_k, int n, int ld,
                    int has_relu, const float *__restrict__ lamL, const float *__restrict__ lamU,
                    const float *__restrict__ nuU, const float *__restrict__ bias_below, int *__restrict__ status,
                    float q_scale, float lo_scale) {
    pdl_trigger();
    pdl_wait();
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_warps) return;
    const int chunks = (n_k + kRowsPerWarp - 1) / kRowsPerWarp;
    const long long grp = w / chunks;                  // (box, side)
    const int i0 = (int)(w % chunks) * kRowsPerWarp;
    const int b = (int)(grp >> 1);
    const int upper = (int)(grp & 1);
    const long long r0 = grp * n_k + i0;               // row of neuron i0
    const float *ll = lamL + (size_t)b * ld, *lu = lamU + (size_t)b * ld, *nu = nuU + (size_t)b * ld;
    float dacc[kRowsPerWarp];
#pragma unroll
    for (int rr = 0; rr < kRowsPerWarp; ++rr) dacc[rr] = 0.0f;
    bool out_of_range = false;
    // eight consecutive columns per lane: 16-byte stores of halves (row pitches are multiples of 32 elements)
    for (int t = lane * 8; t < ld; t += 256) {
        float bz[8], la[8], ua[8], na[8];
        {
            const float4 y0 = *reinterpret_cast<const float4 *>(bias_below + t);
            const float4 y1 = *reinterpret_cast<const float4 *>(bias_below + t + 4);
            bz[0] = y0.x; bz[1] = y0.y; bz[2] = y0.z; bz[3] = y0.w; bz[4] = y1.x; bz[5] = y1.y; bz[6] = y1.z; bz[7] = y1.w;
        }
        if (has_relu) {
            const float4 l0 = *reinterpret_cast<const float4 *>(ll + t), l1 = *reinterpret_cast<const float4 *>(ll + t + 4);
            const float4 u0 = *reinterpret_cast<const float4 *>(lu + t), u1 = *reinterpret_cast<const float4 *>(lu + t + 4);
            const float4 n0 = *reinterpret_cast<const float4 *>(nu + t), n1 = *reinterpret_cast<const float4 *>(nu + t + 4);
            la[0] = l0.x; la[1] = l0.y; la[2] = l0.z; la[3] = l0.w; la[4] = l1.x; la[5] = l1.y; la[6] = l1.z; la[7] = l1.w;
            ua[0] = u0.x; ua[1] = u0.y; ua[2] = u0.z; ua[3] = u0.w; ua[4] = u1.x; ua[5] = u1.y; ua[6] = u1.z; ua[7] = u1.w;
            na[0] = n0.x; na[1] = n0.y; na[2] = n0.z; na[3] = n0.w; na[4] = n1.x; na[5] = n1.y; na[6] = n1.z; na[7] = n1.w;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) { la[e] = ua[e] = 1.0f; na[e] = 0.0f; }
        }
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            if (i0 + rr >= n_k) break;
            float c[8], q[8];
            const float *wrow = Wk + (size_t)(i0 + rr) * ldw_k + t;
            const float4 x0 = *reinterpret_cast<const float4 *>(wrow);
            const float4 x1 = *reinterpret_cast<const float4 *>(wrow + 4);
            c[0] = x0.x; c[1] = x0.y; c[2] = x0.z; c[3] = x0.w; c[4] = x1.x; c[5] = x1.y; c[6] = x1.z; c[7] = x1.w;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                q[e] = 0.0f;
                if (t + e < n) {
                    const bool nonneg = (c[e] >= 0.0f);
                    const bool use_lower = upper ? !nonneg : nonneg;
                    q[e] = c[e] * (use_lower ? la[e] : ua[e]);
                    if (!use_lower) dacc[rr] = fmaf(c[e], na[e], dacc[rr]);
                }
            }
            uint32_t ph[4], pl[4];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                __half h[2], l[2];
#pragma unroll
                for (int z = 0; z < 2; ++z) {
                    dacc[rr] = fmaf(q[e + z], bz[e + z], dacc[rr]);
                    const float x = q[e + z] * q_scale;       // a power of two
                    out_of_range |= !(fabsf(x) <= 60000.0f);
                    h[z] = __float2half_rn(x);
                    l[z] = __float2half_rn((x - __half2float(h[z])) * lo_scale);
                }
                ph[e >> 1] = (uint32_t)__half_as_ushort(h[0]) | ((uint32_t)__half_as_ushort(h[1]) << 16);
                pl[e >> 1] = (uint32_t)__half_as_ushort(l[0]) | ((uint32_t)__half_as_ushort(l[1]) << 16);
            }
            CERT_ST(*reinterpret_cast<uint4 *>(Q_hi + (size_t)(r0 + rr) * ld + t), make_uint4(ph[0], ph[1], ph[2], ph[3]));
            CERT_ST(*reinterpret_cast<uint4 *>(Q_lo + (size_t)(r0 + rr) * ld + t), make_uint4(pl[0], pl[1], pl[2], pl[3]));
        }
    }
#pragma unroll
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const float tot = warp_sum16(dacc[rr]);
        if (lane == 0 && i0 + rr < n_k) CERT_ST(d[r0 + rr], bias_k[i0 + rr] + tot);
    }
    if (__any_sync(0xffffffffu, out_of_range) && lane == 0) atomicOr(status, 2);
}

typedef CUresult (*EncodeTiledFn16)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);
EncodeTiledFn16 g_encode16 = nullptr;

template <int EPI, bool ONEPASS>
void launch_one16(int pairs, const CUtensorMap &ah, const CUtensorMap &al, const CUtensorMap &bh,
                  const CUtensorMap &bl, const CUtensorMap &oh, const CUtensorMap &ol, const TcArgs &args,
                  int smem_bytes, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(pairs * 2), 1, 1);
    cfg.blockDim = dim3(kThreads16, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    cudaLaunchKernelEx(&cfg, gemm_tc16_kernel<EPI, ONEPASS>, ah, al, bh, bl, oh, ol, args);
}

template <int EPI, bool ONEPASS>
bool allow_smem16() {
    return cudaFuncSetAttribute(gemm_tc16_kernel<EPI, ONEPASS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kTcSmemMax) == cudaSuccess;
}

}  // namespace

bool tc16_prepare_kernels() {
    if (!g_encode16) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn) {
            cudaGetLastError();
            return false;
        }
        g_encode16 = reinterpret_cast<EncodeTiledFn16>(fn);
    }
    if (!allow_smem16<TC_EPI_RELU_SKIP, false>() || !allow_smem16<TC_EPI_RELU, false>() ||
        !allow_smem16<TC_EPI_REUSE, false>() || !allow_smem16<TC_EPI_CONCRETIZE, false>() ||
        !allow_smem16<TC_EPI_RELU_SKIP, true>() || !allow_smem16<TC_EPI_RELU, true>() ||
        !allow_smem16<TC_EPI_CONCRETIZE, true>()) {
        cudaGetLastError();
        return false;
    }
    return true;
}

bool tc16_make_map(TcMap *m, const __half *base, long long inner, long long outer, long long pitch_elems,
                   int box_inner, int box_outer) {
    if (!g_encode16) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * sizeof(__half)};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = g_encode16(reinterpret_cast<CUtensorMap *>(m), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
                            const_cast<__half *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

Tc16Plan tc16_tile_plan(int N, int n_tiles) {
    Tc16Plan p;
    p.n_tiles = n_tiles > 0 ? n_tiles : (N + 255) / 256;
    // 32-column units spread over the tiles: the first tiles take one unit more than the last n_narrow ones
    const int units = (N + 31) / 32;
    int b = (units + p.n_tiles - 1) / p.n_tiles * 32;
    p.bn = b;
    p.n_narrow = (b / 32) * p.n_tiles - units;
    if (b < 64) p.n_narrow = 0;           // a 32-column tile cannot lose a unit
    if (p.n_narrow >= p.n_tiles) p.n_narrow = 0;
    const int stage_bytes = 2 * kATileBytes + 2 * (b / 2) * BKH * 2;
    const int fixed = kEpiBytes16 + (int)sizeof(Barriers16) + 1024;
    int st = (kTcSmemMax - fixed) / stage_bytes;
    p.stages = st > 8 ? 8 : st;
    int cols = 32;
    while (cols < 2 * b) cols *= 2;
    p.tmem_cols = cols;
    p.smem_bytes = p.stages * stage_bytes + fixed;
    return p;
}

void launch_gemm_tc16(int epi, bool one_pass, int pairs, const TcMap &a_hi, const TcMap &a_lo, const TcMap &b_hi,
                      const TcMap &b_lo, const TcMap &o_hi, const TcMap &o_lo, const TcArgs &args, int smem_bytes,
                      cudaStream_t st) {
    const CUtensorMap &ah = reinterpret_cast<const CUtensorMap &>(a_hi);
    const CUtensorMap &al = reinterpret_cast<const CUtensorMap &>(a_lo);
    const CUtensorMap &bh = reinterpret_cast<const CUtensorMap &>(b_hi);
    const CUtensorMap &bl = reinterpret_cast<const CUtensorMap &>(b_lo);
    const CUtensorMap &oh = reinterpret_cast<const CUtensorMap &>(o_hi);
    const CUtensorMap &ol = reinterpret_cast<const CUtensorMap &>(o_lo);
    const bool skip = args.add_hi || args.add_identity;
    if (one_pass) {
        if (epi == TC_EPI_RELU && skip) launch_one16<TC_EPI_RELU_SKIP, true>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else if (epi == TC_EPI_RELU) launch_one16<TC_EPI_RELU, true>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else launch_one16<TC_EPI_CONCRETIZE, true>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        return;
    }
    if (epi == TC_EPI_RELU && skip) launch_one16<TC_EPI_RELU_SKIP, false>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
    else if (epi == TC_EPI_RELU) launch_one16<TC_EPI_RELU, false>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
    else if (epi == TC_EPI_REUSE) launch_one16<TC_EPI_REUSE, false>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
    else launch_one16<TC_EPI_CONCRETIZE, false>(pairs, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
}

void launch_init_expr16(const LayerDev &Lk, const LayerDev &Lb, int batch, __half *Q_hi, __half *Q_lo, float *d,
                        int *status, float q_scale, float lo_scale, cudaStream_t st) {
    const long long n_warps = 2LL * batch * ((Lk.n_out + kRowsPerWarp - 1) / kRowsPerWarp);
    launch_chained(expr_start16_kernel, dim3((unsigned)ceil_div_ll(n_warps, 8)), dim3(256), 0, st, Lk.W, Lk.ld_in,
                   Lk.bias_n, Q_hi, Q_lo, d, n_warps, Lk.n_out, Lb.n_out, Lb.ld_out, Lb.relu_after, Lb.lamL, Lb.lamU, Lb.nuU,
                   Lb.bias_n, status, q_scale, lo_scale);
}

}  // namespace cert
