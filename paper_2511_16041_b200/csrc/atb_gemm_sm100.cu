// atb_gemm: C = dequant(A_bfp16) x B_bf16 with asymmetric tile buffering (Section 3), sm_100a.
//
// One persistent CTA per SM walks output tiles of T_MC x T_N (bands of 16 tile rows, odd bands with the
// columns backwards, K upwards in one tile and downwards in the next: tile_coords, serpentine_k - each
// wave of tiles starts on what the wave before it left in the L2).  Per K-step (output-stationary
// schedule of Section 3.1) the T_K x T_N tile of B is brought into shared memory ONCE and
// rho = T_MC / T_MA slabs of A are streamed through it; the FP32 accumulator of the whole
// T_MC x T_N tile lives in tensor memory and is written out once, after K / T_K steps.
//
// Warp roles (736 threads):
//   warp 0      TMA producer of B tiles
//   warp 1      UMMA issuer (one elected lane) and owner of the TMEM allocation
//   warps 2-5   epilogue: tcgen05.ld -> round to bf16 -> swizzled shared-memory box -> TMA store
//   warps 6-21  dequantisers, in 2 or 4 groups that take the slabs (bundles of thin slabs) in turn: raw slab -> bf16,
//               K-major, 128-byte-swizzled operand in shared memory (exact: m * 2^(E-133) has at
//               most 7 significant bits)
//   warp 22     TMA producer of raw BFP16 A slabs (int8 mantissas + uint8 exponents); a warp of its
//               own, so that a full B ring never holds back the slabs the dequantisers wait for
// Rings, all guarded by mbarriers with bounded waits:
//   B tiles          (n_b_stages)    producer -> UMMA          (freed by tcgen05.commit)
//   raw A slabs      (n_raw_stages)  producer -> dequantisers  (freed by the dequantisers)
//   bf16 A groups    (n_groups x 128 rows) dequantisers -> UMMA (freed by tcgen05.commit)
//   accumulators     (acc_bufs x T_MC/128 row groups in TMEM)  UMMA -> epilogue
// The UMMA shape is always 128 x T_N x 16.  A slab of T_MA < 128 rows is the unit of loading; the
// 128 / T_MA consecutive slabs that fill one 128-row operand group are converted and signalled as
// one bundle (see Cfg::BUNDLE).
#include <algorithm>
#include <cmath>

#include "atb_gemm_device.cuh"

namespace {

// Set by a kernel whose bounded wait expired: (role << 8) | barrier kind.
__device__ unsigned int g_gemm_error_flag = 0;

template <int T_MA, int T_MC, int T_K, int T_N>
struct Cfg {
    static constexpr int SLAB_ROWS = T_MA;
    static constexpr int G = T_MC / 128;                       // 128-row groups per output tile
    static constexpr int RHO = T_MC / T_MA;                    // slabs per K-step
    static constexpr int SLABS = RHO;                          // (per 64-column round, the name the shared roles use)
    static constexpr int SPG = (T_MA < 128) ? 128 / T_MA : 1;  // slabs per group
    static constexpr int GPS = (T_MA > 128) ? T_MA / 128 : 1;  // groups per slab
    static constexpr int N_MMA = T_N > 256 ? 256 : T_N;        // UMMA N extent; T_N / N_MMA instructions side by side
    static constexpr int N_CHUNKS = T_N / N_MMA;
    static constexpr uint32_t B_BYTES = T_K * T_N * 2;
    static constexpr uint32_t B_BOX_BYTES = T_K * 128;         // one 64-column box of B
    // T_K is the depth of a B tile.  A always moves in units of kKA = 64 columns - raw slabs of
    // T_MA x 64, converted operand groups of 128 x 64 (one 128-byte swizzle row per row) - so a K-step
    // of T_K = 128 is one B tile and KH = 2 rounds of slabs: the conversion pipeline (slab size, groups,
    // hand-overs per FLOP) is the same for every T_K, only the B ring's grain and the B barriers per
    // FLOP change.
    static constexpr int KH = T_K / kKA;
    static constexpr uint32_t GROUP_BYTES = 128 * kKA * 2;
    static constexpr uint32_t KHALF_BYTES = 128 * 128;         // 128 rows x 64 bf16
    static constexpr uint32_t RAW_MANT_BYTES = T_MA * kKA;
    static constexpr uint32_t RAW_EXP_BYTES = T_MA * kKA / 8;
    static constexpr uint32_t RAW_BYTES = RAW_MANT_BYTES + RAW_EXP_BYTES;
    static constexpr int SLOTS_PER_ROW = kKA / 16;             // a slot = 2 blocks = 16 mantissa bytes
    static constexpr int SLOTS = T_MA * SLOTS_PER_ROW;
    static constexpr int DQ_GROUPS = dq_groups(T_MA, T_K, T_N);
    static constexpr int GROUP_WARPS = kDequantWarps / DQ_GROUPS;
    static constexpr int GROUP_THREADS = GROUP_WARPS * 32;
    static constexpr int DQ_ITERS = (SLOTS + GROUP_THREADS - 1) / GROUP_THREADS;
    static constexpr int ROWS_PER_ITER = GROUP_THREADS / SLOTS_PER_ROW;
    // ring depths (compile-time: every ring index below folds to constants)
    static constexpr RingPlan PLAN = plan_single(T_MA, T_MC, T_K, T_N);
    static constexpr int NB = PLAN.nb, NG = PLAN.ng, NR = PLAN.nr;
    // Thin slabs (T_MA < 128) are converted in bundles of SPG: a dequantiser group takes the SPG slabs
    // of one 128-row operand group per barrier round trip and signals the group once, so the fixed cost
    // of a round (waits, proxy fence, arrivals, the issuer's wait and commit) is paid per 128 rows
    // whatever T_MA is (a shallow raw ring may force smaller bundles: slab_bundle).  Bundles, not slabs,
    // are dealt to the dequantiser groups in turn; a raw-slab barrier must stay with one group, hence
    // lcm(depth, groups * bundle) of them.
    static constexpr int BUNDLE = slab_bundle(SPG, NR, DQ_GROUPS);   // slabs per bundle
    static constexpr int SPB = SPG / BUNDLE;                          // bundles (dequantised stages) per operand group
    static constexpr int ND = (T_MA <= 128) ? NG * SPB : NG / GPS;   // dequantised stages
    static constexpr int LR = ring_bars(NR, DQ_GROUPS * BUNDLE), LD = ring_bars(ND, DQ_GROUPS);
    static_assert(NR % BUNDLE == 0 && LR % BUNDLE == 0 && DQ_GROUPS * BUNDLE <= LR && LD % SPB == 0, "bundles");
    static constexpr int ACC_BUFS = PLAN.acc_bufs, TMEM_COLS = PLAN.tmem_cols;
    static_assert(DQ_GROUPS == PLAN.dqg, "plan");
};

// ---------------------------------------------------------------------------------------------
// SPLIT: partial tiles over K ranges go to an FP32 workspace.  QOUT: C is written as BFP16 planes
// (the C format of the paper's all-BFP16 configurations, Section 6.1) by a quantising epilogue.
template <int T_MA, int T_MC, int T_K, int T_N, bool SPLIT, bool QOUT = false>
__global__ void __launch_bounds__(kThreads, 1)
atb_gemm_kernel(const __grid_constant__ CUtensorMap tm_mant, const __grid_constant__ CUtensorMap tm_exp,
                const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_c,
                const GemmParams p) {
    using C = Cfg<T_MA, T_MC, T_K, T_N>;
    extern __shared__ uint8_t smem_raw[];

    // ---- carve shared memory (1024-byte aligned base: required by the 128-byte swizzle) ----
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t b_base = smem_base;
    const uint32_t deq_base = b_base + C::NB * C::B_BYTES;
    constexpr uint32_t raw_off = C::NB * C::B_BYTES + C::NG * C::GROUP_BYTES;
    const uint32_t raw_base = smem_base + raw_off;
    // epilogue staging: one 32-row x 64-column bf16 box (4 KB, 128-byte swizzle) per epilogue warp
    constexpr uint32_t stage_off = (raw_off + C::NR * C::RAW_BYTES + 1023u) & ~1023u;
    constexpr uint32_t bar_off = stage_off + 4u * kEpilogueBoxBytes;
    const uint32_t bar_base = smem_base + bar_off;          // 8-byte mbarriers
    constexpr int n_acc = C::ACC_BUFS * C::G;
    // barrier indices
    const uint32_t b_full = bar_base, b_empty = b_full + 8 * C::NB;
    const uint32_t raw_full = b_empty + 8 * C::NB, raw_empty = raw_full + 8 * C::LR;
    const uint32_t deq_full = raw_empty + 8 * C::LR, deq_empty = deq_full + 8 * C::LD;
    const uint32_t acc_full = deq_empty + 8 * C::LD, acc_empty = acc_full + 8 * n_acc;
    const uint32_t misc = acc_empty + 8 * n_acc;             // [0]: TMEM base, [1]: abort flag
    volatile uint32_t* const misc_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + (misc - smem_base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Ctx cx{misc_gen + 1, p.error_flag};

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::NB; ++i) { mbar_init(b_full + 8 * i, 1); mbar_init(b_empty + 8 * i, 1); }
        for (int i = 0; i < C::LR; ++i) { mbar_init(raw_full + 8 * i, 1); mbar_init(raw_empty + 8 * i, C::GROUP_WARPS); }
        for (int i = 0; i < C::LD; ++i) { mbar_init(deq_full + 8 * i, C::GROUP_WARPS); mbar_init(deq_empty + 8 * i, 1); }
        for (int i = 0; i < n_acc; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 4); }
        misc_gen[1] = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_mant);
        prefetch_tensormap(&tm_exp);
        prefetch_tensormap(&tm_b);
        prefetch_tensormap(&tm_c);
    }
    if (warp == 1) {
        tmem_alloc(misc, static_cast<uint32_t>(C::TMEM_COLS));
        tmem_relinquish();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = misc_gen[0];
#ifdef ATB_PROFILE
    const long long prof_c0 = clock64();
    const uint64_t prof_t0 = global_timer_ns();
#endif

    const int total_items = p.m_tiles * p.n_tiles * (SPLIT ? p.splits : 1);

    if (warp == 0) {
        // ================================ TMA producer: B tiles ========================
        if (elect_one()) {
            Ring rb;
            bool ok = true;
            int it = 0;
            for (int item = blockIdx.x; ok && item < total_items; item += gridDim.x, ++it) {
                const WorkItem w = work_item<SPLIT>(item, p);
                for (int k0 = w.k_begin; ok && k0 < w.k_end; ++k0) {
                    const int k = serpentine_k(it, k0, w.k_begin, w.k_end);
                    if (!(ok = wait_bar_spin(cx, b_empty + 8 * rb.stage, rb.phase ^ 1u, 0x001))) break;
                    const uint32_t fb = b_full + 8 * rb.stage;
                    mbar_arrive_expect_tx(fb, C::B_BYTES);
#pragma unroll
                    for (int j = 0; j < T_N / 64; ++j)
                        tma_load_2d(b_base + rb.stage * C::B_BYTES + j * C::B_BOX_BYTES, &tm_b,
                                    w.nt * T_N + j * 64, k * T_K, fb);
                    rb.advance(C::NB);
                }
            }
        }
    } else if (warp == kAProducerWarp) {
        // ================================ TMA producer: raw A slabs ====================
        if (elect_one()) {
            int item = blockIdx.x;
            a_producer_role<C>(cx, &tm_mant, &tm_exp, raw_full, raw_empty, raw_base,
                               [&](int, int& row0, int& k_begin, int& k_end) {
                                   if (item >= total_items) return false;
                                   const WorkItem w = work_item<SPLIT>(item, p);
                                   row0 = w.mt * T_MC; k_begin = w.k_begin; k_end = w.k_end;
                                   item += gridDim.x;
                                   return true;
                               });
        }
    } else if (warp == 1) {
        // ================================ UMMA issuer =================================
        if (elect_one()) {
            constexpr uint32_t idesc = umma_idesc_bf16_f32(128, C::N_MMA, false, true);
            Ring rb;
            Cursor<C::ND, C::LD> rd;
            int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < total_items; item += gridDim.x, ++it) {
                const WorkItem w = work_item<SPLIT>(item, p);
                const int acc_buf = it % C::ACC_BUFS;
                const uint32_t acc_phase = static_cast<uint32_t>(it / C::ACC_BUFS) & 1u;
                for (int k = w.k_begin; ok && k < w.k_end; ++k) {
                    if (!(ok = wait_bar_spin(cx, b_full + 8 * rb.stage, rb.phase, 0x101))) break;
                    const uint32_t bs = b_base + rb.stage * C::B_BYTES;
#pragma unroll
                    for (int h = 0; h < C::KH; ++h) {         // 64-column rounds of this B tile
                    for (int g = 0; g < C::G; ++g) {
                        const int acc = acc_buf * C::G + g;
                        if (k == w.k_begin && h == 0 && !(ok = wait_bar_spin(cx, acc_empty + 8 * acc, acc_phase ^ 1u, 0x102))) break;
                        int group_slot;
                        if (T_MA <= 128) {
                            for (int i = 0; ok && i < C::SPB; ++i)
                                ok = wait_bar_spin(cx, deq_full + 8 * (rd.bar + i), rd.phase, 0x103);
                            if (!ok) break;
                            group_slot = rd.buf() / C::SPB;
                        } else {
                            if ((g % C::GPS) == 0 && !(ok = wait_bar_spin(cx, deq_full + 8 * rd.bar, rd.phase, 0x103))) break;
                            group_slot = rd.buf() * C::GPS + (g % C::GPS);
                        }
                        tcgen05_fence_after_sync();
                        const uint32_t as = deq_base + group_slot * C::GROUP_BYTES;
                        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * T_N);
#pragma unroll
                        for (int nc = 0; nc < C::N_CHUNKS; ++nc) {
#pragma unroll
                            for (int kk = 0; kk < kKA / 16; ++kk) {
                                const uint64_t a_desc = umma_smem_desc_sw128(as + kk * 32, 16, 1024);
                                const uint64_t b_desc = umma_smem_desc_sw128(bs + nc * (C::N_MMA / 64) * C::B_BOX_BYTES + (h * 4 + kk) * 2048,
                                                                             C::B_BOX_BYTES, 1024);
                                umma_f16_ss(d_tmem + nc * C::N_MMA, a_desc, b_desc, idesc, (k > w.k_begin || h > 0 || kk > 0) ? 1u : 0u);
                            }
                        }
                        if (T_MA <= 128) {
                            for (int i = 0; i < C::SPB; ++i) umma_commit(deq_empty + 8 * (rd.bar + i));
                            rd.template advance<C::SPB>();
                        } else if ((g % C::GPS) == C::GPS - 1) {
                            umma_commit(deq_empty + 8 * rd.bar);
                            rd.template advance<1>();
                        }
                        if (k == w.k_end - 1 && h == C::KH - 1) umma_commit(acc_full + 8 * acc);
                    }
                    if (!ok) break;
                    }
                    if (!ok) break;
                    umma_commit(b_empty + 8 * rb.stage);
                    rb.advance(C::NB);
                }
            }
        }
    } else if (warp < kFirstDequantWarp) {
        // ================================ epilogue ====================================
        const int q = warp & 3;                       // TMEM lane quadrant this warp may access
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < total_items; item += gridDim.x, ++it) {
            const WorkItem w = work_item<SPLIT>(item, p);
            const int mt = w.mt, nt = w.nt;
            const int acc_buf = it % C::ACC_BUFS;
            const uint32_t acc_phase = static_cast<uint32_t>(it / C::ACC_BUFS) & 1u;
            for (int g = 0; g < C::G; ++g) {
                const int acc = acc_buf * C::G + g;
                if (!(ok = wait_bar(cx, acc_full + 8 * acc, acc_phase, 0x201))) break;
                tcgen05_fence_after_sync();
                const int row0 = mt * T_MC + g * 128 + q * 32;          // first of this warp's 32 rows
                const int col0 = nt * T_N;
                const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(acc * T_N);
                const uint32_t box = smem_base + stage_off + static_cast<uint32_t>(warp - kFirstEpilogueWarp) * kEpilogueBoxBytes;
                if (SPLIT) {
                    // FP32 partial tile -> workspace [split][m_pad][N]: boxes of 32 rows x 32 columns
                    const uint32_t my_row = box + lane * 128;
                    const uint32_t sw = static_cast<uint32_t>(lane & 7);
#pragma unroll 1
                    for (int c = 0; c < T_N / 32; ++c) {
                        if (lane == 0) tma_store_wait_read<0>();
                        __syncwarp();
                        uint32_t v[32];
                        tmem_ld_32x32b_x32(t_addr + c * 32, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + ((static_cast<uint32_t>(j) ^ sw) << 4)),
                                         "r"(v[4 * j]), "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3]) : "memory");
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0 && col0 + c * 32 < p.N) {
                            tma_store_2d(&tm_c, box, col0 + c * 32, w.split * p.m_pad + row0);
                            tma_store_commit();
                        }
                    }
                } else if (QOUT) {
                    epilogue_bfp16<T_N>(&tm_c, t_addr, box, lane, row0, col0, p.M, p.N, p.C_exp, p.c_exp_rows);
                } else {
                    epilogue_bf16<T_N>(&tm_c, p.C, p.ldc, t_addr, box, lane, row0, col0, p.M, p.N);
                }
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty + 8 * acc);
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    } else {
        // ================================ dequantisers ================================
        const int t = (threadIdx.x - kFirstDequantWarp * 32) % C::GROUP_THREADS;
        const int my_group = (threadIdx.x - kFirstDequantWarp * 32) / C::GROUP_THREADS;
        // The dequantisers do not need to know tiles or K-steps: slabs arrive in ring order, so a
        // group just takes every DQ_GROUPS-th slab of this CTA's stream.
        int64_t my_slabs = 0;
        for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
            const WorkItem w = work_item<SPLIT>(item, p);
            my_slabs += static_cast<int64_t>(w.k_end - w.k_begin) * C::KH * C::RHO;
        }
        dequantiser_role<C, false>(cx, t, my_group, warp, lane, my_slabs, raw_full, raw_empty, deq_full, deq_empty, raw_base, deq_base);
    }

    // ---- teardown: on the abort path give copies and MMAs in flight time to land first ----
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
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, static_cast<uint32_t>(C::TMEM_COLS));
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// SPLIT = false: Cout is bf16 C[M][ldc].  SPLIT = true: Cout is the FP32 workspace
// [splits][m_tiles * T_MC][N] that receives one partial tile per (tile, split).
template <int T_MA, int T_MC, int T_K, int T_N, bool SPLIT = false, bool QOUT = false>
atb_status_t launch(const atb::GemmPlan& plan, int64_t M, int64_t N, int64_t K, const int8_t* mant,
                    const uint8_t* exp, const void* B, int64_t ldb, void* Cout, int64_t ldc,
                    int num_sms, unsigned int* error_flag, cudaStream_t stream, int splits = 1,
                    uint8_t* C_exp = nullptr) {
    CUtensorMap tm_mant, tm_exp, tm_b, tm_c;
    const int64_t M_pad = atb::round_up(M, 32);
    if (!make_map_2d(&tm_mant, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, mant, K, M, K, kKA, T_MA, CU_TENSOR_MAP_SWIZZLE_NONE))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the mantissa plane");
    if (!make_map_2d(&tm_exp, CU_TENSOR_MAP_DATA_TYPE_UINT64, 8, exp, M_pad, atb::ceil_div(K, 64), M_pad * 8, T_MA,
                     1, CU_TENSOR_MAP_SWIZZLE_NONE))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the exponent plane");
    if (!make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B, N, K, ldb * 2, 64, T_K, CU_TENSOR_MAP_SWIZZLE_128B))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for B");
    const int64_t m_pad = atb::ceil_div(M, T_MC) * T_MC;
    if (SPLIT) {
        if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Cout, N, splits * m_pad, N * 4, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the split-K workspace");
    } else if (QOUT) {
        if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Cout, N, M, ldc, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the mantissa plane of C");
    } else if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Cout, N, M, ldc * 2, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) {
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for C");
    }

    GemmParams p;
    p.M = M; p.N = N; p.K = K; p.ldc = ldc;
    p.C = static_cast<__nv_bfloat16*>(Cout);
    p.m_tiles = static_cast<int>(atb::ceil_div(M, T_MC));
    p.n_tiles = static_cast<int>(atb::ceil_div(N, T_N));
    p.k_steps = static_cast<int>(atb::ceil_div(K, T_K));
    p.error_flag = error_flag;
    p.splits = splits;
    p.m_pad = static_cast<int>(m_pad);
    p.C_exp = C_exp;
    p.c_exp_rows = M_pad;

    auto kernel = atb_gemm_kernel<T_MA, T_MC, T_K, T_N, SPLIT, QOUT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(plan.smem_bytes));
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int64_t items = static_cast<int64_t>(p.m_tiles) * p.n_tiles * splits;
    const int grid = static_cast<int>(items < num_sms ? items : num_sms);
    kernel<<<grid, kThreads, plan.smem_bytes, stream>>>(tm_mant, tm_exp, tm_b, tm_c, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "gemm launch: %s", cudaGetErrorString(e));
    return ATB_OK;
}

// Split-K reduction: C[m][n] = bf16(sum over splits of the FP32 partials), 8 columns per thread.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ ws, int splits, int64_t m_pad, int64_t M, int64_t N,
                     __nv_bfloat16* __restrict__ C, int64_t ldc) {
    const int64_t vec_per_row = N >> 3;
    const int64_t total = M * vec_per_row;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t m = i / vec_per_row, n = (i - m * vec_per_row) << 3;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int s = 0; s < splits; ++s) {
            const float4* src = reinterpret_cast<const float4*>(ws + (s * m_pad + m) * N + n);
            const float4 a = __ldg(src), b = __ldg(src + 1);
            acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
            acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
        }
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * j], acc[2 * j + 1]);
            o[j] = *reinterpret_cast<uint32_t*>(&b2);
        }
        *reinterpret_cast<uint4*>(C + m * ldc + n) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

struct DeviceInfo {
    bool known = false;
    int cc_major = 0, cc_minor = 0, num_sms = 0;
    unsigned int* error_flag = nullptr;
};
DeviceInfo g_devices[64];
std::mutex g_devices_mutex;

atb_status_t device_info(DeviceInfo** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "device ordinal %d out of range", dev);
    std::lock_guard<std::mutex> lock(g_devices_mutex);
    DeviceInfo& d = g_devices[dev];
    if (!d.known) {
        cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
        cudaDeviceGetAttribute(&d.cc_minor, cudaDevAttrComputeCapabilityMinor, dev);
        cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (d.cc_major == 10 && d.cc_minor == 0) {
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&d.error_flag), g_gemm_error_flag);
            if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        }
        d.known = true;
    }
    *out = &d;
    return ATB_OK;
}

}  // namespace

namespace atb {

static void fill_plan(const RingPlan& pl, GemmPlan* plan) {
    plan->dq_groups = pl.dqg;
    plan->n_b_stages = pl.nb;
    plan->n_groups = pl.ng;
    plan->n_raw_stages = pl.nr;
    plan->acc_bufs = pl.acc_bufs;
    plan->tmem_cols = pl.tmem_cols;
    plan->smem_bytes = pl.smem_bytes;
}

bool plan_gemm(int T_MA, int T_MC, int T_K, int T_N, GemmPlan* plan, bool single_cta) {
    if (T_MA <= 0 || T_MC <= 0 || T_MA > T_MC) return false;
    // On the CTA pair each SM holds 128 rows of the tile: a slab cannot be taller than that, and
    // T_MA = 128 is the pair's symmetric form.
    if (is_pair_tiling(T_MC, T_K, T_N) && T_MA > 128) return false;
    const RingPlan pl = is_pair_tiling(T_MC, T_K, T_N)                            ? plan_pair(T_MA, 512)
                        : (is_stacked_pair_tiling(T_MC, T_K, T_N) && !single_cta) ? plan_pair(T_MA, 256)
                                                                                  : plan_single(T_MA, T_MC, T_K, T_N);
    if (!pl.ok || !(T_MA == 32 || T_MA == 64 || T_MA == 128 || T_MA == 256)) return false;
    fill_plan(pl, plan);
    return true;
}

}  // namespace atb

extern "C" int atb_tiling_supported(int T_MA, int T_MC, int T_K, int T_N) {
    atb::GemmPlan plan;
    return atb::plan_gemm(T_MA, T_MC, T_K, T_N, &plan) ? 1 : 0;
}

extern "C" atb_status_t atb_tiling_plan(int T_MA, int T_MC, int T_K, int T_N, atb_plan_t* out) {
    atb::clear_error();
    if (!out) return atb::fail(ATB_ERR_NULL_POINTER, "out must be non-NULL");
    atb::GemmPlan plan;
    if (T_MA <= 0 || T_MC <= 0 || T_MC % T_MA != 0 || !atb::plan_gemm(T_MA, T_MC, T_K, T_N, &plan))
        return atb::fail(ATB_ERR_BAD_TILING, "tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d) is not supported", T_MA, T_MC, T_K, T_N);
    out->n_b_stages = plan.n_b_stages;
    out->n_raw_stages = plan.n_raw_stages;
    out->n_a_groups = plan.n_groups;
    out->dequant_groups = plan.dq_groups;
    out->acc_buffers = plan.acc_bufs;
    out->tmem_columns = plan.tmem_cols;
    out->smem_bytes = static_cast<int>(plan.smem_bytes);
    return ATB_OK;
}

#define ATB_DISPATCH_TN(TMA_, TMC_, TK_)                                                               \
    switch (T_N) {                                                                                     \
        case 64:  return launch<TMA_, TMC_, TK_, 64>(plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc, dev->num_sms, dev->error_flag, st);  \
        case 128: return launch<TMA_, TMC_, TK_, 128>(plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc, dev->num_sms, dev->error_flag, st); \
        case 256: if constexpr ((TMC_ / 128) * 256 <= 512)                                             \
                      return launch<TMA_, TMC_, TK_, 256>(plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc, dev->num_sms, dev->error_flag, st); \
                  break;                                                                               \
        case 512: if constexpr ((TMC_ / 128) * 512 <= 512 && TK_ == 64)                                \
                      return launch<TMA_, TMC_, TK_, 512>(plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc, dev->num_sms, dev->error_flag, st); \
                  break;                                                                               \
    }                                                                                                  \
    break;

#define ATB_DISPATCH_TK(TMA_, TMC_)                      \
    if (T_K == 64) { ATB_DISPATCH_TN(TMA_, TMC_, 64) }   \
    else { ATB_DISPATCH_TN(TMA_, TMC_, 128) }

extern "C" atb_status_t atb_gemm(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                 const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                 const void* B_bf16_dev, int64_t ldb, void* C_bf16_dev, int64_t ldc,
                                 void* stream) {
    atb::clear_error();
    if (!A_mant_dev || !A_exp_dev || !B_bf16_dev || !C_bf16_dev)
        return atb::fail(ATB_ERR_NULL_POINTER, "A_mant_dev, A_exp_dev, B_bf16_dev and C_bf16_dev must be non-NULL");
    if (M < 1 || N < 1 || K < 16 || K % 16 != 0 || N % 8 != 0)
        return atb::fail(ATB_ERR_BAD_SHAPE, "need M >= 1, N >= 8 with N %% 8 == 0, K >= 16 with K %% 16 == 0 (got %lld, %lld, %lld)",
                         (long long)M, (long long)N, (long long)K);
    if (M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30))
        return atb::fail(ATB_ERR_BAD_SHAPE, "dimensions above 2^30 are not supported");
    if (ldb < N || ldc < N || ldb % 8 != 0 || ldc % 8 != 0)
        return atb::fail(ATB_ERR_BAD_SHAPE, "ldb=%lld and ldc=%lld must be >= N and multiples of 8", (long long)ldb, (long long)ldc);
    if (!atb::aligned16(A_mant_dev) || !atb::aligned16(A_exp_dev) || !atb::aligned16(B_bf16_dev) || !atb::aligned16(C_bf16_dev))
        return atb::fail(ATB_ERR_MISALIGNED, "all device pointers must be 16-byte aligned");
    atb::GemmPlan plan;
    if (T_MA <= 0 || T_MC <= 0 || T_MC % T_MA != 0 || !atb::plan_gemm(T_MA, T_MC, T_K, T_N, &plan))
        return atb::fail(ATB_ERR_BAD_TILING, "tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d) is not supported", T_MA, T_MC, T_K, T_N);
    DeviceInfo* dev = nullptr;
    atb_status_t st_dev = device_info(&dev);
    if (st_dev != ATB_OK) return st_dev;
    if (dev->cc_major != 10 || dev->cc_minor != 0)
        return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d; this library runs on 10.0 only", dev->cc_major, dev->cc_minor);
    if (static_cast<int64_t>(atb::ceil_div(M, T_MC)) * atb::ceil_div(N, T_N) > (1ll << 30))
        return atb::fail(ATB_ERR_BAD_SHAPE, "too many output tiles");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (atb::is_pair_tiling(T_MC, T_K, T_N))
        return atb::launch_gemm_pair(T_MA, 512, plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc,
                                     dev->num_sms, dev->error_flag, stream);
    if (atb::is_stacked_pair_tiling(T_MC, T_K, T_N)) {
        // Two 128 x 256 tiles, one above the other, on a CTA pair that shares their B tiles; a problem of one
        // tile row has nothing to share and runs on single CTAs.
        if (M > 128)
            return atb::launch_gemm_pair(T_MA, 256, plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_bf16_dev, ldc,
                                         dev->num_sms, dev->error_flag, stream);
        if (!atb::plan_gemm(T_MA, T_MC, T_K, T_N, &plan, true))
            return atb::fail(ATB_ERR_BAD_TILING, "tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d) is not supported", T_MA, T_MC, T_K, T_N);
    }

    switch (T_MC) {
        case 128:
            switch (T_MA) {
                case 32:  ATB_DISPATCH_TK(32, 128)
                case 64:  ATB_DISPATCH_TK(64, 128)
                case 128: ATB_DISPATCH_TK(128, 128)
            }
            break;
        case 256:
            switch (T_MA) {
                case 32:  ATB_DISPATCH_TK(32, 256)
                case 64:  ATB_DISPATCH_TK(64, 256)
                case 128: ATB_DISPATCH_TK(128, 256)
                case 256: ATB_DISPATCH_TK(256, 256)
            }
            break;
        case 384:                       // three 128-row groups: rho = 3, 6, 12
            switch (T_MA) {
                case 32:  ATB_DISPATCH_TK(32, 384)
                case 64:  ATB_DISPATCH_TK(64, 384)
                case 128: ATB_DISPATCH_TK(128, 384)
            }
            break;
    }
    return atb::fail(ATB_ERR_BAD_TILING, "no kernel for tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d)", T_MA, T_MC, T_K, T_N);
}

extern "C" atb_status_t atb_device_status(void* stream) {
    atb::clear_error();
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaStreamSynchronize: %s", cudaGetErrorString(e));
    unsigned int flag = 0;
    e = cudaMemcpyFromSymbol(&flag, g_gemm_error_flag, sizeof flag);
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaMemcpyFromSymbol: %s", cudaGetErrorString(e));
    if (flag != 0) {
        const unsigned int zero = 0;
        cudaMemcpyToSymbol(g_gemm_error_flag, &zero, sizeof zero);
        return atb::fail(ATB_ERR_DEVICE_TIMEOUT, "a GEMM kernel gave up a bounded wait (code 0x%03x)", flag);
    }
    flag = atb::take_cfg_error_flag();
    if (flag != 0)
        return atb::fail(ATB_ERR_DEVICE_TIMEOUT, "a precision-configuration GEMM kernel gave up a bounded wait (code 0x%03x)", flag);
    return ATB_OK;
}

// ---------------------------------------------------------------------------------------------
// Split-K
// ---------------------------------------------------------------------------------------------
namespace {

bool splitk_tiling_ok(int T_MA, int T_MC, int T_K, int T_N) {
    return T_K == 64 && (T_MC == 128 || T_MC == 256) && (T_N == 128 || T_N == 256) &&
           (T_MA == 64 || T_MA == 128) && T_MA <= T_MC;
}

atb_status_t splitk_validate(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N, int splits) {
    if (M < 1 || N < 8 || N % 8 != 0 || K < 16 || K % 16 != 0 || M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30))
        return atb::fail(ATB_ERR_BAD_SHAPE, "need M >= 1, N %% 8 == 0, K %% 16 == 0 (got %lld, %lld, %lld)", (long long)M, (long long)N, (long long)K);
    if (!splitk_tiling_ok(T_MA, T_MC, T_K, T_N))
        return atb::fail(ATB_ERR_BAD_TILING, "split-K supports T_K = 64, T_MC in {128, 256}, T_N in {128, 256}, T_MA in {64, 128}");
    if (splits < 1 || splits > 64 || splits > atb::ceil_div(K, T_K))
        return atb::fail(ATB_ERR_BAD_SHAPE, "splits=%d must be in [1, min(64, ceil(K / T_K))]", splits);
    // the partial tiles are addressed by a 32-bit TMA row coordinate split * roundup(M, T_MC) + row
    if (static_cast<int64_t>(splits) * atb::round_up(M, T_MC) > 0x7FFFFFFFll)
        return atb::fail(ATB_ERR_BAD_SHAPE, "splits * roundup(M, T_MC) = %lld exceeds 2^31 - 1",
                         (long long)(static_cast<int64_t>(splits) * atb::round_up(M, T_MC)));
    return ATB_OK;
}

}  // namespace

extern "C" size_t atb_gemm_splitk_workspace_bytes(int64_t M, int64_t N, int T_MC, int splits) {
    if (M < 1 || N < 1 || T_MC < 1 || splits < 1) return 0;
    return static_cast<size_t>(splits) * static_cast<size_t>(atb::ceil_div(M, T_MC) * T_MC) * static_cast<size_t>(N) * sizeof(float);
}

namespace atb {

// Runs the split-K GEMM with partials in `ws` (device, at least the documented size) and reduces.
atb_status_t gemm_splitk_with_workspace(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                        const int8_t* mant, const uint8_t* exp, const void* B, int64_t ldb,
                                        void* C, int64_t ldc, int splits, float* ws, void* stream) {
    GemmPlan plan;
    if (!plan_gemm(T_MA, T_MC, T_K, T_N, &plan, true))      // split-K runs on single CTAs
        return fail(ATB_ERR_BAD_TILING, "tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d) is not supported", T_MA, T_MC, T_K, T_N);
    DeviceInfo* dev = nullptr;
    atb_status_t st_dev = device_info(&dev);
    if (st_dev != ATB_OK) return st_dev;
    if (dev->cc_major != 10 || dev->cc_minor != 0)
        return fail(ATB_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d; this library runs on 10.0 only", dev->cc_major, dev->cc_minor);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    atb_status_t rc = ATB_ERR_BAD_TILING;
#define ATB_SPLIT_CASE(TMA_, TMC_, TN_)                                                                         \
    if (T_MA == TMA_ && T_MC == TMC_ && T_N == TN_)                                                             \
        rc = launch<TMA_, TMC_, 64, TN_, true>(plan, M, N, K, mant, exp, B, ldb, ws, 0, dev->num_sms, dev->error_flag, st, splits);
    ATB_SPLIT_CASE(64, 128, 128) ATB_SPLIT_CASE(128, 128, 128) ATB_SPLIT_CASE(64, 128, 256) ATB_SPLIT_CASE(128, 128, 256)
    ATB_SPLIT_CASE(64, 256, 128) ATB_SPLIT_CASE(128, 256, 128) ATB_SPLIT_CASE(64, 256, 256) ATB_SPLIT_CASE(128, 256, 256)
#undef ATB_SPLIT_CASE
    if (rc != ATB_OK) return rc;
    const int64_t vecs = M * (N / 8);
    const int blocks = static_cast<int>(std::min<int64_t>((vecs + 255) / 256, static_cast<int64_t>(dev->num_sms) * 8));
    splitk_reduce_kernel<<<blocks, 256, 0, st>>>(ws, splits, ceil_div(M, T_MC) * T_MC, M, N,
                                                 static_cast<__nv_bfloat16*>(C), ldc);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ATB_ERR_CUDA, "split-K reduce launch: %s", cudaGetErrorString(e));
    return ATB_OK;
}

}  // namespace atb

// ---------------------------------------------------------------------------------------------
// GEMM with a quantising epilogue: C in BFP16
// ---------------------------------------------------------------------------------------------
extern "C" atb_status_t atb_gemm_bfp16_out(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                           const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                           const void* B_bf16_dev, int64_t ldb,
                                           int8_t* C_mant_dev, uint8_t* C_exp_dev, void* stream) {
    atb::clear_error();
    if (!A_mant_dev || !A_exp_dev || !B_bf16_dev || !C_mant_dev || !C_exp_dev)
        return atb::fail(ATB_ERR_NULL_POINTER, "all device pointers must be non-NULL");
    if (M < 1 || N < 16 || N % 16 != 0 || K < 16 || K % 16 != 0 || M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30))
        return atb::fail(ATB_ERR_BAD_SHAPE, "need M >= 1, N %% 16 == 0, K %% 16 == 0 (got %lld, %lld, %lld)", (long long)M, (long long)N, (long long)K);
    if (ldb < N || ldb % 8 != 0) return atb::fail(ATB_ERR_BAD_SHAPE, "ldb=%lld must be >= N and a multiple of 8", (long long)ldb);
    const bool pair = atb::is_pair_tiling(T_MC, T_K, T_N) && (T_MA == 64 || T_MA == 128);
    // (T_MA, 128, 128, 256): two stacked tiles on a CTA pair where there is more than one tile row, as in atb_gemm
    const bool stacked = atb::is_stacked_pair_tiling(T_MC, T_K, T_N) && (T_MA == 64 || T_MA == 128);
    if (!pair && !stacked && !splitk_tiling_ok(T_MA, T_MC, T_K, T_N))
        return atb::fail(ATB_ERR_BAD_TILING, "the quantising epilogue supports T_MA in {64, 128} with T_K = 64, T_MC in {128, 256}, T_N in {128, 256}; with (T_MC, T_K, T_N) = (256, 64, 512); and with (128, 128, 256)");
    if (!atb::aligned16(A_mant_dev) || !atb::aligned16(A_exp_dev) || !atb::aligned16(B_bf16_dev) || !atb::aligned16(C_mant_dev) ||
        !atb::aligned16(C_exp_dev))
        return atb::fail(ATB_ERR_MISALIGNED, "all device pointers must be 16-byte aligned");
    atb::GemmPlan plan;
    const bool stacked_pair = stacked && M > 128;
    if (!atb::plan_gemm(T_MA, T_MC, T_K, T_N, &plan, /*single_cta=*/!stacked_pair))
        return atb::fail(ATB_ERR_BAD_TILING, "tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d) is not supported", T_MA, T_MC, T_K, T_N);
    DeviceInfo* dev = nullptr;
    atb_status_t st_dev = device_info(&dev);
    if (st_dev != ATB_OK) return st_dev;
    if (dev->cc_major != 10 || dev->cc_minor != 0)
        return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d; this library runs on 10.0 only", dev->cc_major, dev->cc_minor);
    if (pair || stacked_pair)
        return atb::launch_gemm_pair(T_MA, pair ? 512 : 256, plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb, C_mant_dev, N,
                                     dev->num_sms, dev->error_flag, stream, C_exp_dev);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define ATB_QOUT_CASE(TMA_, TMC_, TK_, TN_)                                                                      \
    if (T_MA == TMA_ && T_MC == TMC_ && T_K == TK_ && T_N == TN_)                                                \
        return launch<TMA_, TMC_, TK_, TN_, false, true>(plan, M, N, K, A_mant_dev, A_exp_dev, B_bf16_dev, ldb,  \
                                                         C_mant_dev, N, dev->num_sms, dev->error_flag, st, 1, C_exp_dev);
    ATB_QOUT_CASE(64, 128, 64, 128) ATB_QOUT_CASE(128, 128, 64, 128) ATB_QOUT_CASE(64, 128, 64, 256) ATB_QOUT_CASE(128, 128, 64, 256)
    ATB_QOUT_CASE(64, 256, 64, 128) ATB_QOUT_CASE(128, 256, 64, 128) ATB_QOUT_CASE(64, 256, 64, 256) ATB_QOUT_CASE(128, 256, 64, 256)
    ATB_QOUT_CASE(64, 128, 128, 256) ATB_QOUT_CASE(128, 128, 128, 256)        // one tile row of the stacked tiling
#undef ATB_QOUT_CASE
    return atb::fail(ATB_ERR_BAD_TILING, "no kernel for tiling (T_MA=%d, T_MC=%d, T_K=%d, T_N=%d)", T_MA, T_MC, T_K, T_N);
}

extern "C" atb_status_t atb_gemm_splitk(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                        const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                        const void* B_bf16_dev, int64_t ldb, void* C_bf16_dev, int64_t ldc,
                                        int splits, float* workspace_dev, size_t workspace_bytes, void* stream) {
    atb::clear_error();
    if (!A_mant_dev || !A_exp_dev || !B_bf16_dev || !C_bf16_dev || !workspace_dev)
        return atb::fail(ATB_ERR_NULL_POINTER, "all device pointers, including the workspace, must be non-NULL");
    atb_status_t v = splitk_validate(M, N, K, T_MA, T_MC, T_K, T_N, splits);
    if (v != ATB_OK) return v;
    if (ldb < N || ldc < N || ldb % 8 != 0 || ldc % 8 != 0)
        return atb::fail(ATB_ERR_BAD_SHAPE, "ldb=%lld and ldc=%lld must be >= N and multiples of 8", (long long)ldb, (long long)ldc);
    if (!atb::aligned16(A_mant_dev) || !atb::aligned16(A_exp_dev) || !atb::aligned16(B_bf16_dev) ||
        !atb::aligned16(C_bf16_dev) || !atb::aligned16(workspace_dev))
        return atb::fail(ATB_ERR_MISALIGNED, "all device pointers must be 16-byte aligned");
    if (workspace_bytes < atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits))
        return atb::fail(ATB_ERR_BUFFER_TOO_SMALL, "workspace of %zu bytes is smaller than the %zu needed", workspace_bytes,
                         atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits));
    return atb::gemm_splitk_with_workspace(M, N, K, T_MA, T_MC, T_K, T_N, A_mant_dev, A_exp_dev, B_bf16_dev, ldb,
                                           C_bf16_dev, ldc, splits, workspace_dev, stream);
}

extern "C" int atb_select_splits(int64_t M, int64_t N, int64_t K, int T_MC, int T_K, int T_N) {
    if (M < 1 || N < 1 || K < 1 || T_MC < 1 || T_K < 1 || T_N < 1) return 1;
    const int64_t tiles = atb::ceil_div(M, T_MC) * atb::ceil_div(N, T_N);
    const int64_t k_steps = atb::ceil_div(K, T_K);
    // Fill the 148 SMs once, keep at least 8 K-steps per split, and stop where the FP32 partials
    // (written and read once each) would cost more than the GEMM itself saves.
    int best = 1;
    double best_t = 1e300;
    for (int s = 1; s <= 32; s *= 2) {
        if (s > 1 && k_steps / s < 8) break;
        const double waves = std::ceil(static_cast<double>(tiles * s) / 148.0);
        const double t_gemm = waves * (static_cast<double>(k_steps) / s) * (2.0 * T_MC * T_N * T_K / 8192.0 / 0.8);   // cycles
        const double t_part = s > 1 ? (2.0 * s * M * N * 4.0) / (3.0e12 / 1.4e9) : 0.0;                             // cycles at ~3 TB/s
        const double t = t_gemm + t_part + (s > 1 ? 8000.0 : 0.0);
        if (t < best_t) { best_t = t; best = s; }
    }
    return best;
}

// ---------------------------------------------------------------------------------------------
// Split-K without a caller workspace and without any allocation
// ---------------------------------------------------------------------------------------------
// The FP32 partial tiles go to this fixed array instead of caller memory.  It is part of the
// library image: every GPU on which the library's module gets loaded sets the 64 MiB aside until
// the process exits, whether or not this entry point is ever called.
static __device__ __align__(256) float g_splitk_scratch[ATB_NOALLOC_SCRATCH_BYTES / sizeof(float)];

namespace {

// In host code `g_splitk_scratch` is only a handle for the runtime, not an address a kernel can
// use; the device address has to be asked for, per device, with that device current.
float* g_scratch_ptr[64] = {};
std::mutex g_scratch_mutex;

atb_status_t scratch_address(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "device ordinal %d out of range", dev);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_splitk_scratch);
        if (e != cudaSuccess || !ptr)
            return atb::fail(ATB_ERR_CUDA, "cudaGetSymbolAddress(split-K scratch): %s", cudaGetErrorString(e));
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return ATB_OK;
}

}  // namespace

extern "C" atb_status_t atb_gemm_splitk_noalloc(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                                const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                                const void* B_bf16_dev, int64_t ldb, void* C_bf16_dev, int64_t ldc,
                                                int splits, void* stream) {
    atb::clear_error();
    if (!A_mant_dev || !A_exp_dev || !B_bf16_dev || !C_bf16_dev)
        return atb::fail(ATB_ERR_NULL_POINTER, "A_mant_dev, A_exp_dev, B_bf16_dev and C_bf16_dev must be non-NULL");
    atb_status_t v = splitk_validate(M, N, K, T_MA, T_MC, T_K, T_N, splits);
    if (v != ATB_OK) return v;
    if (ldb < N || ldc < N || ldb % 8 != 0 || ldc % 8 != 0)
        return atb::fail(ATB_ERR_BAD_SHAPE, "ldb=%lld and ldc=%lld must be >= N and multiples of 8", (long long)ldb, (long long)ldc);
    if (!atb::aligned16(A_mant_dev) || !atb::aligned16(A_exp_dev) || !atb::aligned16(B_bf16_dev) || !atb::aligned16(C_bf16_dev))
        return atb::fail(ATB_ERR_MISALIGNED, "all device pointers must be 16-byte aligned");
    const size_t need = atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits);
    if (need > static_cast<size_t>(ATB_NOALLOC_SCRATCH_BYTES))
        return atb::fail(ATB_ERR_BUFFER_TOO_SMALL,
                         "splits * roundup(M, T_MC) * N * 4 = %zu bytes of partial sums exceed the built-in scratch of %zu bytes; "
                         "use fewer splits or atb_gemm_splitk with a workspace of your own",
                         need, static_cast<size_t>(ATB_NOALLOC_SCRATCH_BYTES));
    float* scratch = nullptr;
    v = scratch_address(&scratch);
    if (v != ATB_OK) return v;
    return atb::gemm_splitk_with_workspace(M, N, K, T_MA, T_MC, T_K, T_N, A_mant_dev, A_exp_dev, B_bf16_dev, ldb,
                                           C_bf16_dev, ldc, splits, scratch, stream);
}

#ifdef ATB_PROFILE
// Diagnostic build only: wait-cycle counters of the single-CTA kernels (16 values), read and cleared.
extern "C" int atb_debug_read_wait_cycles(unsigned long long* out16) { return read_wait_cycles(out16); }
#endif
