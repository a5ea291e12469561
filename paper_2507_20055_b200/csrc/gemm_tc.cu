// Affine back-step on the 5th-generation tensor cores (tcgen05), fp32-accurate
// through a three-term TF32 split, with the ReLU back-step or the
// concretisation fused into the epilogue.
//
//   P = Q * W_j                    (Section 4.3, Matmul rewrite of the traversal step)
//   Q' = P+ * lam_a + P- * lam_b   (replace_lower/upper through the ReLU below,
//   d += P(+/-) . nuU + Q' . b       clamp form of Section 4.3), or
//   bound = P+ . l0 + P- . u0 + d  (map(simplify_lower/upper) at the input)
//
// Every fp32 operand x is held as hi = tf32(x) and lo = tf32(x - hi); the
// product is hi*hi + lo*hi + hi*lo accumulated in fp32 in tensor memory.
//
// Persistent kernel.  A work tile is a row panel (128 rows per CTA) times a
// column tile of W_j; the thread that owns a row (its TMEM lane) adds that
// tile's share of the row constant in a register and writes it to the tile's
// slot: no atomics, fixed summation order.
// CTAS = 2: two CTAs of a cluster share a 256-row panel.  Each stages its own
// 128 rows of Q and its own half of the W_j tile, the leader issues
// tcgen05.mma.cta_group::2 over both halves (every B byte is staged and read
// once per pair, not once per CTA), and each CTA runs the epilogue of its own
// 128 accumulator rows.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (one TMEM lane quarter each); results leave through a
// swizzled shared-memory slab and TMA stores.
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace cert {

namespace {

constexpr int BM = 128;                  // rows per CTA
constexpr int BK = 32;                   // floats of K per stage: one 128-byte swizzle row
constexpr int kThreads = 192;
constexpr int kATileBytes = BM * BK * 4;
constexpr int kSlabBytes = 32 * 128;     // 32 rows x 32 floats per epilogue warp and output array
constexpr int kEpiBytes = 4 * 2 * kSlabBytes;

struct __align__(8) Barriers {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// Group g (a CTA, or a CTA pair) works on tiles g, g + n_groups, ...; tile t covers row panel
// t / n_tiles and column tile t % n_tiles, so the groups that run at the same time share row
// panels and the A operand is fetched from DRAM once.
template <int EPI, int CTAS>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
               const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
               const __grid_constant__ CUtensorMap map_o_hi, const __grid_constant__ CUtensorMap map_o_lo,
               const TcArgs a) {
    constexpr bool kBand = (EPI == TC_EPI_RELU_BAND || EPI == TC_EPI_CONCRETIZE_BAND || EPI == TC_EPI_RELU_BAND_SKIP);
    constexpr bool kRelu = (EPI == TC_EPI_RELU || EPI == TC_EPI_RELU_SKIP || EPI == TC_EPI_RELU_BAND ||
                            EPI == TC_EPI_RELU_BAND_SKIP);
    constexpr bool kSkip = (EPI == TC_EPI_RELU_SKIP || EPI == TC_EPI_RELU_BAND_SKIP);
    constexpr bool kStores = kRelu;
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    // tiles are aligned to 1024 bytes (a whole swizzle pattern)
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.bn;
    const int BNL = BN / CTAS;                 // rows of the W_j tile this CTA stages
    const int stages = a.stages;
    const uint32_t b_tile_bytes = (uint32_t)BNL * BK * 4;
    const uint32_t stage_bytes = 2 * kATileBytes + 2 * b_tile_bytes;
    uint8_t *epi_smem = smem + (size_t)stages * stage_bytes;
    Barriers *bars = reinterpret_cast<Barriers *>(epi_smem + kEpiBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (a.K + BK - 1) / BK;
    const int n_tiles = a.n_tiles;
    int total_tiles = a.total_tiles;
    const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const int group = CTAS == 2 ? (int)cluster_id_x() : (int)blockIdx.x;
    const int n_groups = CTAS == 2 ? (int)num_clusters_x() : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->acc_full[i], 1);
            mbar_init(&bars->acc_empty[i], 4 * CTAS);
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        if (CTAS == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&bars->tmem_base)),
                         "r"((uint32_t)a.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&bars->tmem_base)),
                         "r"((uint32_t)a.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();      // the peer's barriers exist before anything arrives on them
    tcgen05_fence_after();
    pdl_wait();                             // everything above needed nothing from the kernel before
    // a re-run that turned out not to be needed has no tiles: every role falls through to the common exit
    if (a.run_if && *reinterpret_cast<const volatile int *>(a.run_if) == 0) total_tiles = 0;
    const uint32_t tmem_base = bars->tmem_base;
    volatile uint32_t *abort_flag = &bars->abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            int armed = 0;      // stage loads issued so far
            const int bands = kBand ? a.n_bands : 1;
            for (int t = group; t < total_tiles && ok; t += n_groups) {
                const int row0 = (t / (n_tiles * bands)) * (BM * CTAS) + (int)rank * BM;
                const int col0 = (t % n_tiles) * BN + (int)rank * BNL;
                // banded form: the K window of this tile's band, clipped to the map (whole map rows = whole k-blocks)
                int kb_lo = 0, kb_hi = num_kb, a_k0 = 0;
                if (kBand) {
                    const int first = (t / n_tiles) % bands - a.band_o_shift;      // first map row of the window
                    const int per_row = a.band_row_in / BK;
                    kb_lo = (first < 0 ? -first : 0) * per_row;
                    const int rows_in = a.band_h_in - first < a.band_rin ? a.band_h_in - first : a.band_rin;
                    kb_hi = rows_in * per_row;
                    a_k0 = first * a.band_row_in;
                }
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(&bars->empty[s], phase ^ 1) || *abort_flag) { ok = false; break; }
                    uint8_t *st = smem + (size_t)s * stage_bytes;
                    // the leader's barrier counts the bytes of every CTA of the group
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[s], stage_bytes * CTAS);
                    const uint32_t bar = CTAS == 2 ? map_to_cta(smem_u32(&bars->full[s]), 0) : smem_u32(&bars->full[s]);
                    const int kx = kb * BK;
                    tma_load_2d<CTAS>(smem_u32(st), &map_a_hi, bar, a_k0 + kx, row0);
                    tma_load_2d<CTAS>(smem_u32(st + kATileBytes), &map_a_lo, bar, a_k0 + kx, row0);
                    tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes), &map_b_hi, bar, kx, col0);
                    tma_load_2d<CTAS>(smem_u32(st + 2 * kATileBytes + b_tile_bytes), &map_b_lo, bar, kx, col0);
                    ++armed;
                    if (++s == stages) { s = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(a.status, 1);
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
        // ------------------------------------------------------------ MMA issuer (the leader CTA of a pair)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                   ((uint32_t)((BM * CTAS) >> 4) << 24);
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            int lt = 0;
            for (int t = group; t < total_tiles && ok; t += n_groups, ++lt) {
                const int acc = lt & 1;
                const uint32_t acc_phase = (lt >> 1) & 1;
                if (!mbar_wait(&bars->acc_empty[acc], acc_phase ^ 1) || *abort_flag) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                int kb_lo = 0, kb_hi = num_kb;
                if (kBand) {
                    const int first = (t / n_tiles) % a.n_bands - a.band_o_shift;
                    const int per_row = a.band_row_in / BK;
                    kb_lo = (first < 0 ? -first : 0) * per_row;
                    kb_hi = (a.band_h_in - first < a.band_rin ? a.band_h_in - first : a.band_rin) * per_row;
                }
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(&bars->full[s], phase) || *abort_flag) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t st = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t da_hi = make_desc(st);
                    const uint64_t da_lo = make_desc(st + kATileBytes);
                    const uint64_t db_hi = make_desc(st + 2 * kATileBytes);
                    const uint64_t db_lo = make_desc(st + 2 * kATileBytes + b_tile_bytes);
#pragma unroll
                    for (int k = 0; k < BK / 8; ++k) {
                        const uint64_t ko = (uint64_t)(k * 2);   // 8 floats = 32 bytes = 2 x 16-byte units
                        mma_tf32<CTAS>(d_tmem, da_lo + ko, db_hi + ko, idesc, ((kb - kb_lo) | k) ? 1u : 0u);
                        mma_tf32<CTAS>(d_tmem, da_hi + ko, db_lo + ko, idesc, 1u);
                        mma_tf32<CTAS>(d_tmem, da_hi + ko, db_hi + ko, idesc, 1u);
                    }
                    tcgen05_commit<CTAS>(&bars->empty[s]);     // frees the stage (in every CTA) when these MMAs retire
                    if (++s == stages) { s = 0; phase ^= 1; }
                }
                if (ok) tcgen05_commit<CTAS>(&bars->acc_full[acc]);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(a.status, 1);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                       // TMEM lane quarter this warp may read
        uint8_t *slab_hi = epi_smem + (size_t)(warp - 2) * 2 * kSlabBytes;
        uint8_t *slab_lo = slab_hi + kSlabBytes;
        const uint32_t acc_empty_addr0 = CTAS == 2 ? map_to_cta(smem_u32(&bars->acc_empty[0]), 0)
                                                   : smem_u32(&bars->acc_empty[0]);
        bool ok = true;
        int lt = 0;
        const int bands = kBand ? a.n_bands : 1;
        for (int t = group; t < total_tiles && ok; t += n_groups, ++lt) {
            const int nt = t % n_tiles;
            const int band = kBand ? (t / n_tiles) % bands : 0;
            // first column of the band's window in the (y-major) output row; may be negative at the top of the map
            const int band_col0 = kBand ? (band * a.band_s - a.band_y_shift) * a.band_row_out : 0;
            const long long warp_row0 = (long long)(t / (n_tiles * bands)) * (BM * CTAS) + (int)rank * BM + quarter * 32;
            const long long r = warp_row0 + lane;
            const bool row_ok = r < a.M;
            const long long rr = row_ok ? r : 0;
            const int b = (int)(rr / (2LL * a.n_k));
            const int upper = (int)((rr / a.n_k) & 1);
            const size_t relax_row = (size_t)b * a.ld_n;
            float dacc = 0.0f;
            int own = -1;                  // kSkip: the column of the row's own neuron (unit coefficient), if it joins
            if (kSkip && a.add_identity) {
                own = (int)(rr % a.n_k);
                if (kBand) {
                    // channel-major neuron index -> its column in the y-major row
                    const int hw = a.band_h_out * a.band_w_out;
                    const int ch = own / hw, y = (own - ch * hw) / a.band_w_out, x = own % a.band_w_out;
                    own = (y * a.band_c_out + ch) * a.band_w_out + x;
                }
            }
            const int acc = lt & 1;
            const uint32_t acc_phase = (lt >> 1) & 1;
            if (!mbar_wait(&bars->acc_full[acc], acc_phase) || *abort_flag) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
            for (int c0 = 0; c0 < BN; c0 += 32) {
                int col0 = nt * BN + c0;
                if (kBand) {
                    if (col0 >= a.band_s * a.band_row_out) break;
                    col0 += band_col0;
                    if (col0 < 0 || col0 >= a.ld_n) continue;    // a map row above or below the map: no such neurons
                } else if (col0 >= a.ld_n) {
                    break;                                   // warp-uniform; ld_n is a multiple of 32
                }
                uint32_t v[32];
                // a residual connection ends on these neurons: its waiting coefficients for the warp's 32 rows x 32
                // columns are requested before the accumulator is read, four rows (128-byte lines) per instruction:
                // load i brings 16-byte piece lane % 8 of row 4 i + lane / 8
                float4 ch[kSkip ? 8 : 1], cl[kSkip ? 8 : 1];
                const bool joins = kSkip && a.add_hi != nullptr;
                if (kSkip && joins) {
                    const float4 z4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        long long rw = warp_row0 + 4 * i + (lane >> 3);
                        if (rw >= a.M) rw = 0;
                        const size_t o = (size_t)rw * a.ld_n + col0 + (lane & 7) * 4;
                        ch[i] = __ldg(reinterpret_cast<const float4 *>(a.add_hi + o));
                        cl[i] = a.add_lo ? __ldg(reinterpret_cast<const float4 *>(a.add_lo + o)) : z4;
                    }
                }
                __syncwarp();
                tmem_ld32(t_addr + (uint32_t)c0, v);
                tmem_ld_wait();
                if (kRelu) {
                    // the slab is free again once the previous chunk's stores have read it
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                    const uint32_t row_hi = smem_u32(slab_hi) + (uint32_t)lane * 128u;
                    const uint32_t row_lo = smem_u32(slab_lo) + (uint32_t)lane * 128u;
                    if (kSkip && joins) {
                        // through the (free) slab to the lane that owns the row; a lane then reads and rewrites
                        // only its own row
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const uint32_t rw = (uint32_t)(4 * i + (lane >> 3));
                            const uint32_t off = rw * 128u + ((((uint32_t)lane & 7u) ^ (rw & 7u)) << 4);
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(slab_hi) + off),
                                         "f"(ch[i].x), "f"(ch[i].y), "f"(ch[i].z), "f"(ch[i].w) : "memory");
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(slab_lo) + off),
                                         "f"(cl[i].x), "f"(cl[i].y), "f"(cl[i].z), "f"(cl[i].w) : "memory");
                        }
                        __syncwarp();
                    }
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const int col = col0 + g * 4;
                        float q[4];
                        const float4 bz = *reinterpret_cast<const float4 *>(a.bias_below + col);
                        if (kSkip) {
                            // the waiting coefficients and the unit coefficient join before the ReLU back-step
                            float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                            if (joins) {
                                const uint32_t swj = (uint32_t)((g ^ (lane & 7)) << 4);
                                float h4[4], l4[4];
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(h4[0]), "=f"(h4[1]),
                                             "=f"(h4[2]), "=f"(h4[3]) : "r"(row_hi + swj) : "memory");
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(l4[0]), "=f"(l4[1]),
                                             "=f"(l4[2]), "=f"(l4[3]) : "r"(row_lo + swj) : "memory");
#pragma unroll
                                for (int e = 0; e < 4; ++e) s4[e] = h4[e] + l4[e];
                            }
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
                            for (int e = 0; e < 4; ++e) q[e] = __uint_as_float(v[g * 4 + e]);
                        }
                        dacc = fmaf(q[0], bz.x, dacc);
                        dacc = fmaf(q[1], bz.y, dacc);
                        dacc = fmaf(q[2], bz.z, dacc);
                        dacc = fmaf(q[3], bz.w, dacc);
                        // 16-byte chunk g of this lane's slab row, at its 128-byte-swizzle position
                        const uint32_t sw = (uint32_t)((g ^ (lane & 7)) << 4);
                        if (a.split_out) {
                            float h[4], l[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                h[e] = tf32_round(q[e]);
                                l[e] = tf32_round(q[e] - h[e]);
                            }
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(row_hi + sw), "f"(h[0]),
                                         "f"(h[1]), "f"(h[2]), "f"(h[3]) : "memory");
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(row_lo + sw), "f"(l[0]),
                                         "f"(l[1]), "f"(l[2]), "f"(l[3]) : "memory");
                        } else {
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(row_hi + sw), "f"(q[0]),
                                         "f"(q[1]), "f"(q[2]), "f"(q[3]) : "memory");
                        }
                    }
                    fence_async_smem();
                    __syncwarp();
                    // rows past the end of the matrix land in scratch rows of the workspace or are clipped
                    if (lane == 0) {
                        tma_store_2d(&map_o_hi, smem_u32(slab_hi), col0, (int)warp_row0);
                        if (a.split_out) tma_store_2d(&map_o_lo, smem_u32(slab_lo), col0, (int)warp_row0);
                        tma_store_commit();
                    }
                } else if (row_ok) {
                    const float *lrow = a.l0 + relax_row + col0;
                    const float *urow = a.u0 + relax_row + col0;
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
            // This tile's share of the row constant (of the bound, for the concretising
            // epilogue) goes to slot nt; the tile of column 0 also carries the constant so far.
            if (row_ok) {
                float tot = dacc;
                const int slot = band * n_tiles + nt;
                if (slot == 0) {
                    float prev = 0.0f;
                    for (int sidx = 0; sidx < a.n_slots_in; ++sidx) prev += a.d_in[(size_t)sidx * a.slot_stride + r];
                    tot += prev;
                }
                CERT_ST(a.d_out[(size_t)slot * a.slot_stride + r], tot);
            }
        }
        if (kStores && lane == 0) tma_store_wait_all();
        if (!ok && lane == 0) atomicExch(a.status, 1);
    }

    tcgen05_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();      // no CTA leaves while its peer may still reach into it
    if (warp == 1) {
        tcgen05_fence_after();
        if (CTAS == 2)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)a.tmem_cols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)a.tmem_cols)
                         : "memory");
    }
}

// What every wait in the tensor-core kernels does when it runs out, on a barrier nothing arrives on: the wait
// returns after `limit` cycles, the kernel raises the status word and ends normally.
__global__ void bounded_wait_selftest_kernel(int *status, unsigned long long limit) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait_for(&bar, 0, limit)) atomicOr(status, 1);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

template <int EPI, int CTAS>
void launch_one(int groups, const CUtensorMap &ah, const CUtensorMap &al, const CUtensorMap &bh,
                const CUtensorMap &bl, const CUtensorMap &oh, const CUtensorMap &ol, const TcArgs &args,
                int smem_bytes, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(groups * CTAS), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
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
    cudaLaunchKernelEx(&cfg, gemm_tc_kernel<EPI, CTAS>, ah, al, bh, bl, oh, ol, args);
}

}  // namespace

void launch_bounded_wait_selftest(int *status, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status, 200000ull);      // about 0.1 ms
}

bool tc_driver_init() {
    if (g_encode) return true;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return false;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return true;
}

bool tc_prepare_kernels(bool *pair_ok) {
    const void *kernels[] = {
        (const void *)gemm_tc_kernel<TC_EPI_RELU, 1>,                (const void *)gemm_tc_kernel<TC_EPI_RELU, 2>,
        (const void *)gemm_tc_kernel<TC_EPI_CONCRETIZE, 1>,          (const void *)gemm_tc_kernel<TC_EPI_CONCRETIZE, 2>,
        (const void *)gemm_tc_kernel<TC_EPI_RELU_SKIP, 1>,           (const void *)gemm_tc_kernel<TC_EPI_RELU_SKIP, 2>,
        (const void *)gemm_tc_kernel<TC_EPI_RELU_BAND, 1>,           (const void *)gemm_tc_kernel<TC_EPI_RELU_BAND, 2>,
        (const void *)gemm_tc_kernel<TC_EPI_CONCRETIZE_BAND, 1>,     (const void *)gemm_tc_kernel<TC_EPI_CONCRETIZE_BAND, 2>,
        (const void *)gemm_tc_kernel<TC_EPI_RELU_BAND_SKIP, 1>,      (const void *)gemm_tc_kernel<TC_EPI_RELU_BAND_SKIP, 2>,
    };
    for (const void *k : kernels)
        if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
    // can a cluster of two such CTAs be resident?
    *pair_ok = false;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kTcSmemMax;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, gemm_tc_kernel<TC_EPI_RELU, 2>, &cfg) == cudaSuccess)
        *pair_ok = n_clusters >= 1;
    else
        cudaGetLastError();
    return true;
}

bool tc_make_map(TcMap *m, const float *base, long long inner, long long outer, long long pitch_floats,
                 int box_outer) {
    if (!g_encode) return false;
    static_assert(sizeof(TcMap) == sizeof(CUtensorMap), "tensor map size");
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_floats * sizeof(float)};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = g_encode(reinterpret_cast<CUtensorMap *>(m), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                          const_cast<float *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

TcPlan tc_tile_plan(int N, int ctas) {
    TcPlan p;
    p.n_tiles = (N + 255) / 256;
    int b = ((N + p.n_tiles - 1) / p.n_tiles + 31) / 32 * 32;
    p.bn = b;
    const int stage_bytes = 2 * kATileBytes + 2 * (b / ctas) * BK * 4;
    const int fixed = kEpiBytes + (int)sizeof(Barriers) + 1024;   // epilogue slabs, barriers, alignment slack
    int st = (kTcSmemMax - fixed) / stage_bytes;
    p.stages = st > 8 ? 8 : st;
    int cols = 32;
    while (cols < 2 * b) cols *= 2;
    p.tmem_cols = cols;
    p.smem_bytes = p.stages * stage_bytes + fixed;
    return p;
}

void launch_gemm_tc(int epi, int ctas, int groups, const TcMap &a_hi, const TcMap &a_lo, const TcMap &b_hi,
                    const TcMap &b_lo, const TcMap &o_hi, const TcMap &o_lo, const TcArgs &args, int smem_bytes,
                    cudaStream_t st) {
    const CUtensorMap &ah = reinterpret_cast<const CUtensorMap &>(a_hi);
    const CUtensorMap &al = reinterpret_cast<const CUtensorMap &>(a_lo);
    const CUtensorMap &bh = reinterpret_cast<const CUtensorMap &>(b_hi);
    const CUtensorMap &bl = reinterpret_cast<const CUtensorMap &>(b_lo);
    const CUtensorMap &oh = reinterpret_cast<const CUtensorMap &>(o_hi);
    const CUtensorMap &ol = reinterpret_cast<const CUtensorMap &>(o_lo);
    if (epi == TC_EPI_RELU_BAND && (args.add_hi || args.add_identity)) {
        if (ctas == 2) launch_one<TC_EPI_RELU_BAND_SKIP, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else launch_one<TC_EPI_RELU_BAND_SKIP, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        return;
    }
    if (epi == TC_EPI_RELU_BAND || epi == TC_EPI_CONCRETIZE_BAND) {
        if (epi == TC_EPI_RELU_BAND) {
            if (ctas == 2) launch_one<TC_EPI_RELU_BAND, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
            else launch_one<TC_EPI_RELU_BAND, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        } else {
            if (ctas == 2) launch_one<TC_EPI_CONCRETIZE_BAND, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
            else launch_one<TC_EPI_CONCRETIZE_BAND, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        }
        return;
    }
    const bool skip = args.add_hi || args.add_identity;
    if (epi == TC_EPI_RELU && skip) {
        if (ctas == 2) launch_one<TC_EPI_RELU_SKIP, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else launch_one<TC_EPI_RELU_SKIP, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        return;
    }
    if (ctas == 2) {
        if (epi == TC_EPI_RELU) launch_one<TC_EPI_RELU, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else launch_one<TC_EPI_CONCRETIZE, 2>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
    } else {
        if (epi == TC_EPI_RELU) launch_one<TC_EPI_RELU, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
        else launch_one<TC_EPI_CONCRETIZE, 1>(groups, ah, al, bh, bl, oh, ol, args, smem_bytes, st);
    }
}

}  // namespace cert
