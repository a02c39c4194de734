// atb_gemm, CTA-pair kernel (sm_100a): the tiling T_MC = 256, T_N = 512, T_K = 64, described first, and at the
// end of this comment the stacked form of the tiling T_MC = 128, T_N = 256, T_K = 128.
//
// Two CTAs of a cluster share one 256 x 512 output tile through tcgen05.mma cta_group::2:
// CTA r (r = 0, 1) owns rows 128r .. 128r+127 of the tile - it loads, dequantises and feeds that
// half of A, and holds its 128 x 512 FP32 accumulator in its own TMEM (all 512 columns) - and
// supplies half of every 256-column B chunk (columns 128r .. 128r+127) from its own shared
// memory.  This is the B200 counterpart of the array-level sharing of Section 3.2 (Eq. 2): the
// B tile is shared across the two "rows" of the pair, and every dequantised A element feeds
// 512 output columns instead of 256, which halves the dequantiser work per FLOP.
//
// Per K-step (Section 3.1 schedule): each CTA brings in its 64 x 256 half of the B tile once and
// streams 128 / SLAB_ROWS raw A slabs through the dequantisers; the leader CTA (rank 0) issues
// 2 x 4 UMMAs of 256 x 256 x 16.  Barriers the UMMA issuer waits on live in the leader CTA and
// collect arrivals from both CTAs; stage-free barriers are signalled in both CTAs at once by
// tcgen05.commit with a CTA mask.  No TMA load uses multicast.
//
// Warp roles are those of the single-CTA kernel: 0 TMA producer of B, 1 UMMA issuer (active in the
// leader only) + TMEM owner, 2-5 epilogue, 6-21 dequantisers (4 groups of 4 warps), 22 TMA producer of A.
// The epilogue stages C in boxes of 32 x 64 BF16 and writes them out with plain coalesced stores (under
// 32-row slabs: boxes of 32 x 32, which leaves room for a fifth dequantised-operand group).
//
// T_N = 256 (the tiling T_MC = 128, T_K = 128, T_N = 256 on a problem of more than one tile row): the pair
// computes two 128 x 256 tiles, one above the other - CTA r the rows 128r.. of a 256-row stripe - and shares their
// B tiles as above.  Each CTA's accumulator takes 256 of its 512 tensor-memory columns, so successive tiles
// alternate between two accumulators and the epilogue of a tile runs beside the K loop of the next one.  A B stage
// is 128 rows deep and serves two 64-column rounds of A, so that the leader needs both CTAs' operands every
// 512 and their B half-tiles every 1024 tensor cycles, as in the single-CTA 256 x 256 tiling.
#include "atb_gemm_device.cuh"

namespace {

template <int SLAB_ROWS_T, int T_N>
struct PairCfg {
    static_assert(T_N == 512 || T_N == 256, "a pair covers 256 x 512, or two stacked tiles of 128 x 256");
    static constexpr int SLAB_ROWS = SLAB_ROWS_T;              // rows of a raw A slab (T_MA)
    static constexpr int T_K = T_N == 512 ? 64 : 128;          // depth of a B stage
    static constexpr int KH = T_K / kKA;                       // 64-column rounds of A per B stage
    static constexpr int N_MMA = 256, N_CHUNKS = T_N / N_MMA, ROWS = 128;
    // Accumulator slots of 128 rows x 256 columns per CTA, two either way: the two chunks of a 512-wide
    // tile, or two buffers of a 256-wide tile that successive tiles take in turn.
    static constexpr int ACC_BUFS = 2 / N_CHUNKS, N_ACC = 2;
    static constexpr int SLABS = ROWS / SLAB_ROWS;             // slabs per CTA and K-step
    static constexpr int GPS = 1;                              // a slab never spans operand groups here
    static constexpr uint32_t B_BOX_BYTES = T_K * 128;         // 64 columns x T_K rows of bf16
    static constexpr uint32_t B_BYTES = (T_N / 128) * B_BOX_BYTES;   // this CTA's half: 128 columns of every chunk
    static constexpr uint32_t GROUP_BYTES = 128 * kKA * 2;
    static constexpr uint32_t KHALF_BYTES = 128 * 128;
    // The 512-wide tile's drain is on the critical path (tensor memory is full): plain coalesced stores get C out
    // fastest.  The stacked tiles' drain runs beside the next tile's K loop: there the one-instruction TMA store,
    // which takes no issue slots from the dequantisers, is ahead (+2.7 % at K = 2048, +1 % at 4096^3 and 8192^3).
    static constexpr bool DIRECT_STORES = (ATB_EPILOGUE_DIRECT_PAIR != 0) && T_N == 512;
    static constexpr int BOX_COLS = pair_box_cols(SLAB_ROWS, T_N);   // epilogue staging box of a warp: 32 rows x BOX_COLS bf16
    static constexpr uint32_t BOX_BYTES = pair_box_bytes(SLAB_ROWS, T_N);
    static constexpr uint32_t RAW_MANT_BYTES = SLAB_ROWS * kKA;
    static constexpr uint32_t RAW_EXP_BYTES = SLAB_ROWS * kKA / 8;
    static constexpr uint32_t RAW_BYTES = RAW_MANT_BYTES + RAW_EXP_BYTES;
    static constexpr int SLOTS_PER_ROW = kKA / 16;
    static constexpr int SLOTS = SLAB_ROWS * SLOTS_PER_ROW;
    static constexpr int DQ_GROUPS = 4;
    static constexpr int GROUP_WARPS = kDequantWarps / DQ_GROUPS;
    static constexpr int GROUP_THREADS = GROUP_WARPS * 32;
    static constexpr int DQ_ITERS = (SLOTS + GROUP_THREADS - 1) / GROUP_THREADS;
    static constexpr int ROWS_PER_ITER = GROUP_THREADS / SLOTS_PER_ROW;
    // ring depths (compile-time)
    static constexpr RingPlan PLAN = plan_pair(SLAB_ROWS, T_N);
    static constexpr int NB = PLAN.nb, NG = PLAN.ng, NR = PLAN.nr;
    // thin slabs are converted and signalled in bundles, as in atb_gemm_kernel
    static constexpr int BUNDLE = slab_bundle(SLABS, NR, DQ_GROUPS), SPB = SLABS / BUNDLE;
    static constexpr int ND = NG * SPB;                        // dequantised stages
    static constexpr int LR = ring_bars(NR, DQ_GROUPS * BUNDLE), LD = ring_bars(ND, DQ_GROUPS);
    static_assert(NR % BUNDLE == 0 && LR % BUNDLE == 0 && DQ_GROUPS * BUNDLE <= LR && LD % SPB == 0, "bundles");
    static_assert(PLAN.ok && DQ_GROUPS == PLAN.dqg && ACC_BUFS == PLAN.acc_bufs && B_BYTES == 4 * 64 * 128, "plan");
};

struct PairParams {
    int64_t M, N, K, ldc;
    __nv_bfloat16* C;                        // bf16 C[M][ldc] (not used by the quantising epilogue)
    int m_tiles, n_tiles, k_steps;           // tiles (stripes) of 256 x T_N, steps of T_K
    unsigned int* error_flag;
    uint8_t* C_exp;                          // QOUT: exponent plane of C and its padded row count
    int64_t c_exp_rows;
};

// Bounded waits with cluster-scope acquire (the arrivals may come from the peer CTA).
__device__ __forceinline__ bool wait_bar_cl(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
    return wait_bar_t<false, true>(cx, bar, parity, code);
}
__device__ __forceinline__ bool wait_bar_cl_spin(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
    return wait_bar_t<true, true>(cx, bar, parity, code);
}

// QOUT: C is written as BFP16 planes by the quantising epilogue (see atb_gemm_bfp16_out).
template <int SLAB_ROWS, int T_N, bool QOUT = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
atb_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_mant, const __grid_constant__ CUtensorMap tm_exp,
                     const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_c,
                     const PairParams p) {
    using C = PairCfg<SLAB_ROWS, T_N>;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t b_base = smem_base;
    const uint32_t deq_base = b_base + C::NB * C::B_BYTES;
    constexpr uint32_t raw_off = C::NB * C::B_BYTES + C::NG * C::GROUP_BYTES;
    const uint32_t raw_base = smem_base + raw_off;
    constexpr uint32_t stage_off = (raw_off + C::NR * C::RAW_BYTES + 1023u) & ~1023u;
    constexpr uint32_t bar_off = stage_off + 4u * C::BOX_BYTES;
    const uint32_t bar_base = smem_base + bar_off;
    const uint32_t b_full = bar_base, b_empty = b_full + 8 * C::NB;
    const uint32_t raw_full = b_empty + 8 * C::NB, raw_empty = raw_full + 8 * C::LR;
    const uint32_t deq_full = raw_empty + 8 * C::LR, deq_empty = deq_full + 8 * C::LD;
    const uint32_t acc_full = deq_empty + 8 * C::LD, acc_empty = acc_full + 8 * C::N_ACC;
    const uint32_t misc = acc_empty + 8 * C::N_ACC;       // [0]: TMEM base, [1]: abort flag
    volatile uint32_t* const misc_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + (misc - smem_base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    Ctx cx{misc_gen + 1, p.error_flag};

    if (threadIdx.x == 0) {
        // Barriers with arrivals from both CTAs are only used in the leader, but are initialised
        // everywhere so that both CTAs have the same layout.
        for (int i = 0; i < C::NB; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
        for (int i = 0; i < C::LR; ++i) { mbar_init(raw_full + 8 * i, 1); mbar_init(raw_empty + 8 * i, C::GROUP_WARPS); }
        for (int i = 0; i < C::LD; ++i) { mbar_init(deq_full + 8 * i, 2 * C::GROUP_WARPS); mbar_init(deq_empty + 8 * i, 1); }
        for (int i = 0; i < C::N_ACC; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 8); }
        misc_gen[1] = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_mant);
        prefetch_tensormap(&tm_exp);
        prefetch_tensormap(&tm_b);
        prefetch_tensormap(&tm_c);
    }
    if (warp == 1) {
        tmem_alloc_pair(misc, 512u);
        tmem_relinquish_pair();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                      // the peer's barriers exist before anything arrives on them
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = misc_gen[0];
#ifdef ATB_PROFILE
    const long long prof_c0 = clock64();
    const uint64_t prof_t0 = global_timer_ns();
#endif

    const int total_tiles = p.m_tiles * p.n_tiles;
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    if (warp == 0) {
        // ================================ TMA producer: B half-tiles ===================
        if (elect_one()) {
            Ring rb;
            bool ok = true;
            int it = 0;
            for (int tile = cluster_id; ok && tile < total_tiles; tile += n_clusters, ++it) {
                int mt, nt;
                tile_coords(tile, p.m_tiles, p.n_tiles, mt, nt);
                const int colb = nt * T_N + static_cast<int>(rank) * 128;
                for (int k0 = 0; ok && k0 < p.k_steps; ++k0) {
                    const int k = serpentine_k(it, k0, 0, p.k_steps);
                    if (!(ok = wait_bar_cl_spin(cx, b_empty + 8 * rb.stage, rb.phase ^ 1u, 0x001))) break;
                    // both halves of the B tile are credited to the leader's barrier
                    if (leader) mbar_arrive_expect_tx(b_full + 8 * rb.stage, 2 * C::B_BYTES);
                    const uint32_t fb = mapa_shared(b_full + 8 * rb.stage, 0);
#ifdef ATB_PROFILE
                    const long long issue_t0 = clock64();
#endif
#pragma unroll
                    for (int j = 0; j < T_N / 128; ++j)
                        tma_load_2d_pair(b_base + rb.stage * C::B_BYTES + j * C::B_BOX_BYTES, &tm_b,
                                         colb + (j >> 1) * 256 + (j & 1) * 64, k * C::T_K, fb);
#ifdef ATB_PROFILE      // slot 8: cycles this thread spent issuing the loads of B
                    atomicAdd(&g_wait_cycles[blockIdx.x & 255][8], static_cast<unsigned long long>(clock64() - issue_t0));
#endif
                    rb.advance(C::NB);
                }
            }
        }
    } else if (warp == kAProducerWarp) {
        // ================================ TMA producer: raw A slabs ====================
        if (elect_one()) {
            int tile = cluster_id;
            a_producer_role<C>(cx, &tm_mant, &tm_exp, raw_full, raw_empty, raw_base,
                               [&](int, int& row0, int& k_begin, int& k_end) {
                                   if (tile >= total_tiles) return false;
                                   int mt, nt;
                                   tile_coords(tile, p.m_tiles, p.n_tiles, mt, nt);
                                   row0 = mt * 256 + static_cast<int>(rank) * 128; k_begin = 0; k_end = p.k_steps;
                                   tile += n_clusters;
                                   return true;
                               });
        }
    } else if (warp == 1) {
        // ================================ UMMA issuer (leader CTA) ====================
        if (leader && elect_one()) {
            constexpr uint32_t idesc = umma_idesc_bf16_f32(256, C::N_MMA, false, true);
            Ring rb;
            Cursor<C::ND, C::LD> rd;
            bool ok = true;
            if constexpr (T_N == 512) {
            uint32_t acc_phase = 0;
            for (int tile = cluster_id; ok && tile < total_tiles; tile += n_clusters, acc_phase ^= 1u) {
                for (int k = 0; ok && k < p.k_steps; ++k) {
                    if (!(ok = wait_bar_cl_spin(cx, b_full + 8 * rb.stage, rb.phase, 0x101))) break;
                    for (int i = 0; ok && i < C::SPB; ++i)
                        ok = wait_bar_cl_spin(cx, deq_full + 8 * (rd.bar + i), rd.phase, 0x103);
                    if (!ok) break;
                    const uint32_t as = deq_base + (rd.buf() / C::SPB) * C::GROUP_BYTES;
                    const uint32_t bs = b_base + rb.stage * C::B_BYTES;
#pragma unroll
                    for (int nc = 0; nc < C::N_CHUNKS; ++nc) {
                        // both CTAs' epilogues have drained this chunk of the previous tile
                        if (k == 0 && !(ok = wait_bar_cl_spin(cx, acc_empty + 8 * nc, acc_phase ^ 1u, 0x102))) break;
                        tcgen05_fence_after_sync();
#pragma unroll
                        for (int kk = 0; kk < C::T_K / 16; ++kk) {
                            const uint64_t a_desc = umma_smem_desc_sw128(as + kk * 32, 16, 1024);
                            const uint64_t b_desc = umma_smem_desc_sw128(bs + nc * 2 * C::B_BOX_BYTES + kk * 2048,
                                                                         C::B_BOX_BYTES, 1024);
                            umma_f16_ss_pair(tmem_base + nc * C::N_MMA, a_desc, b_desc, idesc, (k > 0 || kk > 0) ? 1u : 0u);
                        }
                        if (k == p.k_steps - 1) umma_commit_pair(acc_full + 8 * nc, 3);
                    }
                    if (!ok) break;
                    for (int i = 0; i < C::SPB; ++i) umma_commit_pair(deq_empty + 8 * (rd.bar + i), 3);
                    rd.template advance<C::SPB>();
                    umma_commit_pair(b_empty + 8 * rb.stage, 3);
                    rb.advance(C::NB);
                }
            }
            } else {
            // two stacked 128 x 256 tiles: one 256-column chunk, successive tiles alternate between two accumulators;
            // a B stage serves KH rounds of A
            int it = 0;
            for (int tile = cluster_id; ok && tile < total_tiles; tile += n_clusters, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = static_cast<uint32_t>(it >> 1) & 1u;
                for (int k = 0; ok && k < p.k_steps; ++k) {
                    if (!(ok = wait_bar_cl_spin(cx, b_full + 8 * rb.stage, rb.phase, 0x101))) break;
                    const uint32_t bs = b_base + rb.stage * C::B_BYTES;
#pragma unroll
                    for (int h = 0; h < C::KH; ++h) {
                        for (int i = 0; ok && i < C::SPB; ++i)
                            ok = wait_bar_cl_spin(cx, deq_full + 8 * (rd.bar + i), rd.phase, 0x103);
                        if (!ok) break;
                        // both CTAs' epilogues have drained this accumulator (the tile before the previous one)
                        if (k == 0 && h == 0 && !(ok = wait_bar_cl_spin(cx, acc_empty + 8 * acc, acc_phase ^ 1u, 0x102))) break;
                        const uint32_t as = deq_base + (rd.buf() / C::SPB) * C::GROUP_BYTES;
                        tcgen05_fence_after_sync();
#pragma unroll
                        for (int kk = 0; kk < kKA / 16; ++kk) {
                            const uint64_t a_desc = umma_smem_desc_sw128(as + kk * 32, 16, 1024);
                            const uint64_t b_desc = umma_smem_desc_sw128(bs + (h * 4 + kk) * 2048, C::B_BOX_BYTES, 1024);
                            umma_f16_ss_pair(tmem_base + acc * C::N_MMA, a_desc, b_desc, idesc, (k > 0 || h > 0 || kk > 0) ? 1u : 0u);
                        }
                        if (k == p.k_steps - 1 && h == C::KH - 1) umma_commit_pair(acc_full + 8 * acc, 3);
                        for (int i = 0; i < C::SPB; ++i) umma_commit_pair(deq_empty + 8 * (rd.bar + i), 3);
                        rd.template advance<C::SPB>();
                    }
                    if (!ok) break;
                    umma_commit_pair(b_empty + 8 * rb.stage, 3);
                    rb.advance(C::NB);
                }
            }
            }
        }
    } else if (warp < kFirstDequantWarp) {
        // ================================ epilogue ====================================
        const int q = warp & 3;
        int it = 0;
        bool ok = true;
        for (int tile = cluster_id; ok && tile < total_tiles; tile += n_clusters, ++it) {
            int mt, nt;
            tile_coords(tile, p.m_tiles, p.n_tiles, mt, nt);
            // accumulator slot of chunk 0 of this tile, and the parity of its barriers' current phase
            const int acc0 = (it % C::ACC_BUFS) * C::N_CHUNKS;
            const uint32_t acc_phase = static_cast<uint32_t>(it / C::ACC_BUFS) & 1u;
            const int row0 = mt * 256 + static_cast<int>(rank) * 128 + q * 32;
            const uint32_t box = smem_base + stage_off + static_cast<uint32_t>(warp - kFirstEpilogueWarp) * C::BOX_BYTES;
            for (int nc0 = 0; nc0 < C::N_CHUNKS; ++nc0) {
                const int nc = acc0 + nc0;
                if (!(ok = wait_bar_cl(cx, acc_full + 8 * nc, acc_phase, 0x201))) break;
                tcgen05_fence_after_sync();
                const int col0 = nt * T_N + nc0 * C::N_MMA;
                const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(nc * C::N_MMA);
                if constexpr (QOUT)
                    epilogue_bfp16<C::N_MMA>(&tm_c, t_addr, box, lane, row0, col0, p.M, p.N, p.C_exp, p.c_exp_rows);
                else
                    epilogue_bf16<C::N_MMA, C::BOX_COLS, C::DIRECT_STORES>(&tm_c, p.C, p.ldc, t_addr, box, lane, row0, col0, p.M, p.N);
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa_shared(acc_empty + 8 * nc, 0));
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    } else {
        // ================================ dequantisers ================================
        const int t = (threadIdx.x - kFirstDequantWarp * 32) % C::GROUP_THREADS;
        const int my_group = (threadIdx.x - kFirstDequantWarp * 32) / C::GROUP_THREADS;
        // slabs arrive in ring order: a group takes every DQ_GROUPS-th slab of this CTA's stream
        int64_t my_slabs = 0;
        for (int tile = cluster_id; tile < total_tiles; tile += n_clusters) my_slabs += static_cast<int64_t>(p.k_steps) * C::KH * C::SLABS;
        dequantiser_role<C, true>(cx, t, my_group, warp, lane, my_slabs, raw_full, raw_empty, deq_full, deq_empty, raw_base, deq_base);
    }

    // ---- teardown: the peer may still arrive on this CTA's barriers until it gets here ----
    if (*cx.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
#ifdef ATB_PROFILE
    if (threadIdx.x == 0) {     // slots 0 / 4: nanoseconds and SM cycles of this CTA's main loop
        atomicAdd(&g_wait_cycles[blockIdx.x & 255][0], static_cast<unsigned long long>(global_timer_ns() - prof_t0));
        atomicAdd(&g_wait_cycles[blockIdx.x & 255][4], static_cast<unsigned long long>(clock64() - prof_c0));
    }
#endif
    cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 512u);
    }
}

template <int SLAB_ROWS, int T_N, bool QOUT = false>
atb_status_t launch_pair_t(const atb::GemmPlan& plan, int64_t M, int64_t N, int64_t K, const int8_t* mant,
                           const uint8_t* exp, const void* B, int64_t ldb, void* Cout, int64_t ldc, int num_sms,
                           unsigned int* error_flag, cudaStream_t stream, uint8_t* C_exp = nullptr) {
    using C = PairCfg<SLAB_ROWS, T_N>;
    CUtensorMap tm_mant, tm_exp, tm_b, tm_c;
    const int64_t M_pad = atb::round_up(M, 32);
    if (!make_map_2d(&tm_mant, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, mant, K, M, K, kKA, SLAB_ROWS, CU_TENSOR_MAP_SWIZZLE_NONE))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the mantissa plane");
    if (!make_map_2d(&tm_exp, CU_TENSOR_MAP_DATA_TYPE_UINT64, 8, exp, M_pad, atb::ceil_div(K, 64), M_pad * 8, SLAB_ROWS, 1,
                     CU_TENSOR_MAP_SWIZZLE_NONE))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the exponent plane");
    if (!make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B, N, K, ldb * 2, 64, C::T_K, CU_TENSOR_MAP_SWIZZLE_128B))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for B");
    if (QOUT) {        // int8 mantissa plane C_mant[M][ldc]: boxes of 32 rows x 64 bytes
        if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Cout, N, M, ldc, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the mantissa plane of C");
    } else if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Cout, N, M, ldc * 2, C::BOX_COLS, 32,
                            C::BOX_COLS == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B)) {
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for C");
    }

    PairParams p;
    p.M = M; p.N = N; p.K = K; p.ldc = ldc;
    p.C = static_cast<__nv_bfloat16*>(Cout);
    p.m_tiles = static_cast<int>(atb::ceil_div(M, 256));
    p.n_tiles = static_cast<int>(atb::ceil_div(N, T_N));
    p.k_steps = static_cast<int>(atb::ceil_div(K, C::T_K));
    p.error_flag = error_flag;
    p.C_exp = C_exp;
    p.c_exp_rows = M_pad;

    auto kernel = atb_gemm_pair_kernel<SLAB_ROWS, T_N, QOUT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(plan.smem_bytes));
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int max_clusters = num_sms / 2;
    const int clusters = static_cast<int>(tiles < max_clusters ? tiles : max_clusters);
    kernel<<<2 * clusters, kThreads, plan.smem_bytes, stream>>>(tm_mant, tm_exp, tm_b, tm_c, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "gemm (pair) launch: %s", cudaGetErrorString(e));
    return ATB_OK;
}

}  // namespace

namespace atb {

atb_status_t launch_gemm_pair(int T_MA, int T_N, const GemmPlan& plan, int64_t M, int64_t N, int64_t K, const int8_t* mant,
                              const uint8_t* exp, const void* B, int64_t ldb, void* C, int64_t ldc, int num_sms,
                              unsigned int* error_flag, void* stream, uint8_t* C_exp) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define ATB_PAIR_CASE(TMA_, TN_, Q_)                                                                                   \
    if (T_MA == TMA_ && T_N == TN_)                                                                                    \
        return launch_pair_t<TMA_, TN_, Q_>(plan, M, N, K, mant, exp, B, ldb, C, ldc, num_sms, error_flag, st, C_exp);
    if (C_exp) {       // BFP16 output: C is the int8 mantissa plane
        ATB_PAIR_CASE(64, 512, true) ATB_PAIR_CASE(128, 512, true) ATB_PAIR_CASE(64, 256, true) ATB_PAIR_CASE(128, 256, true)
        return atb::fail(ATB_ERR_BAD_TILING, "no pair kernel with the quantising epilogue for T_MA=%d, T_N=%d", T_MA, T_N);
    }
    ATB_PAIR_CASE(32, 512, false) ATB_PAIR_CASE(64, 512, false) ATB_PAIR_CASE(128, 512, false)
    ATB_PAIR_CASE(32, 256, false) ATB_PAIR_CASE(64, 256, false) ATB_PAIR_CASE(128, 256, false)
#undef ATB_PAIR_CASE
    return atb::fail(ATB_ERR_BAD_TILING, "no pair kernel for T_MA=%d, T_N=%d", T_MA, T_N);
}

}  // namespace atb

#ifdef ATB_PROFILE
// Diagnostic build only: wait-cycle counters of the CTA-pair kernels (16 values), read and cleared.
extern "C" int atb_debug_read_wait_cycles_pair(unsigned long long* out16) { return read_wait_cycles(out16); }
#endif
