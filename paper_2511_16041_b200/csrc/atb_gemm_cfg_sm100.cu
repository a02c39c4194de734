// atb_gemm_config: the precision configurations the paper evaluates (Section 6.1, Table 2), sm_100a.
//
//   Config 1     A in BF16 (streamed), B in BFP16 (resident), C in BF16
//   Config 2/3   A, B and C in BFP16 (FP32 accumulation here for both)
//
// In both the operand that stays in the core across the rho slabs of a K-step is the BFP16 B tile,
// exactly as in the paper: it is converted ONCE per K-step and every slab of A is multiplied against
// the converted copy (Section 3.1; the "converted copy" term of the buffer column of Table 2).
// B is given as the BFP16 planes of its transpose (N x K, blocks of 8 along K), which is the
// K-major form the UMMA takes for its N-side operand; the dequantised tile is laid out like the
// dequantised A slabs of atb_gemm_kernel and read with a K-major descriptor.
//
// One kernel template, two forms:
//   single CTA  T_MC = 256, T_K = 64, T_N = 256: a CTA holds the 256 x 256 accumulator (all of its tensor
//               memory) and converts both 128-column units of the B tile.
//   CTA pair    T_MC = 512, T_K = 64, T_N = 256 (tcgen05 cta_group::2, M = 256 per instruction): each CTA holds
//               256 rows of the tile and converts ONE unit of the B tile - the tile is shared across the
//               pair (the array-level sharing of Section 3.2, Eq. 2), so a converted B element feeds 512
//               rows and the conversions per FLOP halve.  Barriers the UMMA issuer waits on live in the
//               leader CTA and take arrivals from both; buffers are freed in both CTAs by one
//               tcgen05.commit with a CTA mask.  No TMA load uses multicast.
// Per CTA the streamed operand is the same in both forms: 256 rows of A per K-step in slabs of
// T_MA in {32, 64, 128, 256} rows (rho = 8, 4, 2, 1 per core) - the unit of loading (one TMA box and,
// for BFP16 A, one raw-ring buffer with its own barrier per slab).  The UMMA consumes 128-row operand
// units; slabs thinner than that are gathered (BF16 A: the boxes of a unit land side by side under one
// barrier; BFP16 A: a dequantiser group converts the slabs of a unit as one bundle), a 256-row slab is
// two units under one barrier.  For fixed data the result is bit-identical for every T_MA and for
// both forms.
//   warp 0      TMA producer of raw B units (mantissa box + exponent box)
//   warp 22     TMA producer of A slabs: raw BFP16 (config 2) or BF16 straight into the operand
//               ring, K-major with the 128-byte swizzle (config 1: nothing to convert)
//   warp 1      UMMA issuer (the leader CTA's, on a pair): 128 (256) x 256 x 16, both operands K-major
//   warps 2-5   epilogue (BF16 or quantising BFP16, shared with atb_gemm_kernel)
//   warps 6-21  dequantisers: 4 groups of 4 warps.  The conversion jobs of a K-step - the hand-overs of
//               B that this CTA converts, then the hand-overs of A (config 2) - form one sequence that the groups take
//               in turn, so the work is spread evenly whatever the mix is.
// Barriers, bounded waits and the ring cursors are those of atb_gemm_kernel.
#include "atb_gemm_device.cuh"

namespace {

__device__ unsigned int g_cfg_error_flag = 0;

constexpr int kCfgGroups = 4;                          // dequantiser groups of 4 warps

template <int ROWS>
struct CfgDq {                                         // what dequant_slab needs to know about a slab of ROWS rows
    static constexpr int SLOTS_PER_ROW = 4, SLOTS = ROWS * 4, GROUP_THREADS = 128;
    static constexpr int DQ_ITERS = (SLOTS + GROUP_THREADS - 1) / GROUP_THREADS, ROWS_PER_ITER = 32;
    static constexpr uint32_t KHALF_BYTES = 128 * 128, GROUP_BYTES = 128 * 128;
};

// Barrier pairs of a ring of n buffers whose hand-overs come h per K-step inside a job sequence of
// `ipk` jobs per K-step dealt to kCfgGroups groups in turn: the smallest multiple of n and h for which
// hand-over x and hand-over x + L always fall to the same group (an mbarrier must see its phases
// completed and awaited in order by one group).
constexpr int stream_bars(int n, int h, int ipk) {
    int l = n;
    while (l % h != 0 || ((l / h) * ipk) % kCfgGroups != 0) l += n;
    return l;
}

template <int T_MA, bool A_Q, bool PAIR>
struct CfgK {
    static constexpr int T_K = 64, T_N = 256, ROWS = 256, T_MC = PAIR ? 2 * ROWS : ROWS;
    static_assert(T_MA == 32 || T_MA == 64 || T_MA == 128 || T_MA == 256, "slab height");
    static constexpr int RHO = ROWS / T_MA;                           // slabs of A per K-step and CTA
    static constexpr int SPG = T_MA < 128 ? 128 / T_MA : 1;           // slabs per 128-row operand unit
    static constexpr int GPS = T_MA > 128 ? T_MA / 128 : 1;           // operand units per slab
    static constexpr uint32_t UNIT_BYTES = 128 * 128;                 // 128 rows x 64 bf16
    static constexpr uint32_t RAW_MANT_BYTES = 128 * 64, RAW_BYTES = RAW_MANT_BYTES + 128 * 8;      // a raw B unit
    static constexpr uint32_t SLAB_MANT_BYTES = T_MA * 64, SLAB_RAW_BYTES = SLAB_MANT_BYTES + T_MA * 8;
    static constexpr uint32_t SLAB_BF16_BYTES = T_MA * 128;           // a BF16 slab of A
    static constexpr int UB = PAIR ? 1 : 2;                           // units of the B tile this CTA converts per K-step
    static constexpr int HA = 2 / GPS;                                // hand-overs of A per K-step (a 256-row slab is one)
    static constexpr int JA = A_Q ? HA : 0;                           // ... that are conversion jobs
    static constexpr int IPK = JA + UB;                               // conversion jobs per K-step
    // operand units of A in shared memory: two K-steps; three where BF16 A meets a half-size B ring
    static constexpr int NA = (PAIR && !A_Q) ? 6 : 4;
    static constexpr int NAH = NA / GPS;                              // ... counted in hand-overs
    static constexpr int NAS = A_Q ? (T_MA <= 128 ? 4 * SPG : 2) : 0; // raw A slabs: 512 rows of look-ahead
    static constexpr int LAH = A_Q ? stream_bars(NAH, HA, IPK) : NAH; // barrier pairs of the A operand ring
    static constexpr int LAR = A_Q ? SPG * stream_bars(NAS / SPG, HA, IPK) : 0;   // ... of the raw A ring (bundles of SPG slabs)
    // A converted B tile is held for a whole K-step, by both row groups: three K-steps of tiles where
    // shared memory allows, two otherwise.
    // (config 2 on the pair: six units of A with three or two of B measured 6 % slower than four and four)
    static constexpr int NB = PAIR ? 4 : (A_Q ? 4 : 6), NBR = 4;      // operand / raw units of B
    static constexpr int LB = stream_bars(NB, UB, IPK), LBR = stream_bars(NBR, UB, IPK);
    static constexpr int GROUP_WARPS = 4;
    // Tile-rows per band of the tile walk (tile_coords): the streamed A is the heavier operand here (BF16 in config 1),
    // so a wave should cover few row panels and many column panels of the BFP16 B.
#ifdef ATB_CFG_BAND
    static constexpr int BAND = ATB_CFG_BAND;
#else
    static constexpr int BAND = PAIR ? 4 : 8;
#endif
    static constexpr uint32_t SMEM_BYTES = 1024u + (NA + NB) * UNIT_BYTES + NAS * SLAB_RAW_BYTES + NBR * RAW_BYTES + 1024u +
                                           4u * kEpilogueBoxBytes + 8u * (2 * LAH + 2 * LAR + 2 * LB + 2 * LBR + 4) + 16u;
    static_assert(NB % UB == 0 && LB % UB == 0, "B tiles are whole groups of units");
    static_assert(LAH <= kMaxRingBars && LAR <= kMaxRingBars && LB <= kMaxRingBars && LBR <= kMaxRingBars, "barrier count");
    static_assert(SMEM_BYTES <= kSmemBudget, "shared memory");
};

struct CfgParams {
    int64_t M, N, K, ldc;
    __nv_bfloat16* C;                        // bf16 C[M][ldc] (config 1)
    int m_tiles, n_tiles, k_steps;
    uint8_t* C_exp;
    int64_t c_exp_rows;
    unsigned int* error_flag;
};

// Place of hand-over x of a stream in a ring of N buffers guarded by L barrier pairs (what Cursor
// tracks step by step, computed from x because the dequantisers jump through the job sequence).
template <int N, int L>
struct RingPos {
    int bar, buf;
    uint32_t phase;
    __device__ __forceinline__ explicit RingPos(int64_t x)
        : bar(static_cast<int>(x % L)), buf(static_cast<int>(x % N)), phase(static_cast<uint32_t>(x / L) & 1u) {}
    // the last user of this buffer (hand-over x - N); "before the first" reads as complete on a fresh barrier
    __device__ __forceinline__ int freed_bar() const { return bar < N ? bar - N + L : bar - N; }
    __device__ __forceinline__ uint32_t freed_parity() const { return bar < N ? phase ^ 1u : phase; }
};

// One conversion job of a dequantiser group: hand-over x of a BFP16 stream of slabs of ROWS rows - a
// bundle of 128 / ROWS thin slabs that fill one 128-row operand unit, one 128-row slab, or one 256-row
// slab that fills two units.  NRS raw slabs guarded by LR barrier pairs, NDH hand-overs in the operand
// ring guarded by LD.  On a CTA pair the operand is announced on the leader CTA's barrier (the buffer
// itself stays in this CTA's shared memory and is read by this CTA's tensor core).
template <int ROWS, int NRS, int LR, int NDH, int LD, bool PAIR>
__device__ __forceinline__ bool dequant_job(const Ctx& cx, int64_t x, int t, int lane, uint32_t raw_full, uint32_t raw_empty,
                                            uint32_t deq_full, uint32_t deq_empty, uint32_t raw_base, uint32_t deq_base,
                                            unsigned code) {
    using Dq = CfgDq<ROWS>;
    constexpr int SPG = ROWS < 128 ? 128 / ROWS : 1, GPS = ROWS > 128 ? ROWS / 128 : 1;
    constexpr uint32_t kMant = ROWS * 64, kRaw = kMant + ROWS * 8;
    const DequantLane<Dq> ln(t, ROWS);
    const RingPos<NRS / SPG, LR / SPG> rr(x);      // in bundles: slabs rr.buf * SPG + i, barriers rr.bar * SPG + i
    const RingPos<NDH, LD> rd(x);
    bool ok = true;
#pragma unroll
    for (int i = 0; i < SPG; ++i) ok = ok && wait_bar_t<false, PAIR>(cx, raw_full + 8 * (rr.bar * SPG + i), rr.phase, code | 1u);
    ok = ok && wait_bar_t<false, PAIR>(cx, deq_empty + 8 * rd.freed_bar(), rd.freed_parity(), code | 2u);
    if (!ok) return false;
    const uint32_t dst = deq_base + rd.buf * GPS * Dq::GROUP_BYTES;
    if constexpr (SPG > 1 && SPG * Dq::DQ_ITERS <= 4) {
        dequant_bundle<Dq, SPG>(ln, raw_base + rr.buf * SPG * kRaw, kRaw, kMant, dst, 0, t, ROWS);
    } else {
#pragma unroll
        for (int i = 0; i < SPG; ++i) {
            const uint32_t raw = raw_base + (rr.buf * SPG + i) * kRaw;
            dequant_slab<Dq>(ln, raw, raw + kMant, dst, i * ROWS, t, ROWS);
        }
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        if constexpr (PAIR) {
            // CTA-scope release towards the leader's cluster-scope acquire, as in atb_gemm_pair_kernel: what is
            // published is read by this CTA's own tensor core.  -DATB_PAIR_RELEASE_CLUSTER builds the form the
            // PTX memory model promises to order.
#ifdef ATB_PAIR_RELEASE_CLUSTER
            mbar_arrive_cluster(mapa_shared(deq_full + 8 * rd.bar, 0));
#else
            mbar_arrive_cluster_cta_release(mapa_shared(deq_full + 8 * rd.bar, 0));
#endif
        } else {
            mbar_arrive(deq_full + 8 * rd.bar);
        }
#pragma unroll
        for (int i = 0; i < SPG; ++i) mbar_arrive(raw_empty + 8 * (rr.bar * SPG + i));
    }
    return true;
}

// Frees a buffer (or publishes an accumulator) once the UMMAs issued so far are done: in both CTAs on a pair.
template <bool PAIR>
__device__ __forceinline__ void cfg_commit(uint32_t bar) {
    if constexpr (PAIR) umma_commit_pair(bar, 3);
    else umma_commit(bar);
}

template <int T_MA, bool A_Q, bool C_Q, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
atb_gemm_cfg_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_a_exp,
                    const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_b_exp,
                    const __grid_constant__ CUtensorMap tm_c, const CfgParams p) {
    using C = CfgK<T_MA, A_Q, PAIR>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t a_base = smem_base;                                           // operand units of A
    const uint32_t b_base = a_base + C::NA * C::UNIT_BYTES;                      // operand units of B
    const uint32_t a_raw_base = b_base + C::NB * C::UNIT_BYTES;
    const uint32_t b_raw_base = a_raw_base + C::NAS * C::SLAB_RAW_BYTES;
    constexpr uint32_t stage_off = ((C::NA + C::NB) * C::UNIT_BYTES + C::NAS * C::SLAB_RAW_BYTES + C::NBR * C::RAW_BYTES + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + stage_off + 4u * kEpilogueBoxBytes;
    const uint32_t a_full = bar_base, a_empty = a_full + 8 * C::LAH;
    const uint32_t ar_full = a_empty + 8 * C::LAH, ar_empty = ar_full + 8 * C::LAR;
    const uint32_t b_full = ar_empty + 8 * C::LAR, b_empty = b_full + 8 * C::LB;
    const uint32_t br_full = b_empty + 8 * C::LB, br_empty = br_full + 8 * C::LBR;
    const uint32_t acc_full = br_empty + 8 * C::LBR, acc_empty = acc_full + 8 * 2;
    const uint32_t misc = acc_empty + 8 * 2;                 // [0]: TMEM base, [1]: abort flag
    volatile uint32_t* const misc_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + (misc - smem_base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    constexpr int kCtas = PAIR ? 2 : 1;                      // CTAs whose arrivals the issuer's barriers collect
    Ctx cx{misc_gen + 1, p.error_flag};

    if (threadIdx.x == 0) {
        // On a pair the barriers with arrivals from both CTAs are only used in the leader, but they are
        // initialised everywhere so that both CTAs have the same layout.
        for (int i = 0; i < C::LAH; ++i) { mbar_init(a_full + 8 * i, A_Q ? kCtas * C::GROUP_WARPS : 1); mbar_init(a_empty + 8 * i, 1); }
        for (int i = 0; i < C::LAR; ++i) { mbar_init(ar_full + 8 * i, 1); mbar_init(ar_empty + 8 * i, C::GROUP_WARPS); }
        for (int i = 0; i < C::LB; ++i) { mbar_init(b_full + 8 * i, kCtas * C::GROUP_WARPS); mbar_init(b_empty + 8 * i, 1); }
        for (int i = 0; i < C::LBR; ++i) { mbar_init(br_full + 8 * i, 1); mbar_init(br_empty + 8 * i, C::GROUP_WARPS); }
        for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 4 * kCtas); }
        misc_gen[1] = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_a);
        prefetch_tensormap(&tm_b);
        prefetch_tensormap(&tm_b_exp);
        prefetch_tensormap(&tm_c);
    }
    if (warp == 1) {
        if constexpr (PAIR) { tmem_alloc_pair(misc, 512u); tmem_relinquish_pair(); }
        else { tmem_alloc(misc, 512u); tmem_relinquish(); }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();  // the peer's barriers exist before anything arrives on them
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = misc_gen[0];

    const int total_tiles = p.m_tiles * p.n_tiles;
    const int first_tile = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int tile_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    const int row_off = static_cast<int>(rank) * C::ROWS;    // this CTA's rows inside the tile

    if (warp == 0) {
        // ================================ TMA producer: raw B units ====================
        if (elect_one()) {
            Cursor<C::NBR, C::LBR> rr;
            bool ok = true;
            for (int tile = first_tile; ok && tile < total_tiles; tile += tile_step) {
                int mt, nt;
                tile_coords<C::BAND>(tile, p.m_tiles, p.n_tiles, mt, nt);
                // this CTA's units of the tile: both (single CTA) or unit `rank` (pair)
                const int n0 = nt * C::T_N + (PAIR ? static_cast<int>(rank) * 128 : 0);
                for (int k = 0; ok && k < p.k_steps; ++k) {
                    for (int u = 0; u < C::UB; ++u) {
                        if (!(ok = wait_bar_t<true, PAIR>(cx, br_empty + 8 * rr.freed_bar(), rr.freed_parity(), 0x001))) break;
                        const uint32_t fr = br_full + 8 * rr.bar;
                        const uint32_t dst = b_raw_base + rr.buf() * C::RAW_BYTES;
                        mbar_arrive_expect_tx(fr, C::RAW_BYTES);
                        tma_load_2d(dst, &tm_b, k * C::T_K, n0 + u * 128, fr);
                        tma_load_2d(dst + C::RAW_MANT_BYTES, &tm_b_exp, n0 + u * 128, k, fr);
                        rr.template advance<1>();
                    }
                }
            }
        }
    } else if (warp == kAProducerWarp) {
        // ================================ TMA producer: A units ========================
        if (elect_one()) {
            bool ok = true;
            if constexpr (A_Q) {
                // raw BFP16 slabs of T_MA rows, each with its own buffer and barrier
                Cursor<C::NAS, C::LAR> rr;
                for (int tile = first_tile; ok && tile < total_tiles; tile += tile_step) {
                    int mt, nt;
                    tile_coords<C::BAND>(tile, p.m_tiles, p.n_tiles, mt, nt);
                    const int row0 = mt * C::T_MC + row_off;
                    for (int k = 0; ok && k < p.k_steps; ++k) {
                        for (int sl = 0; sl < C::RHO; ++sl) {
                            if (!(ok = wait_bar_t<true, PAIR>(cx, ar_empty + 8 * rr.freed_bar(), rr.freed_parity(), 0x002))) break;
                            const uint32_t fr = ar_full + 8 * rr.bar;
                            const uint32_t dst = a_raw_base + rr.buf() * C::SLAB_RAW_BYTES;
                            mbar_arrive_expect_tx(fr, C::SLAB_RAW_BYTES);
                            tma_load_2d(dst, &tm_a, k * C::T_K, row0 + sl * T_MA, fr);
                            tma_load_2d(dst + C::SLAB_MANT_BYTES, &tm_a_exp, row0 + sl * T_MA, k, fr);
                            rr.template advance<1>();
                        }
                    }
                }
            } else {
                // BF16 A: the TMA boxes are the UMMA operand (K-major, 128-byte swizzle).  One barrier per
                // hand-over: the slabs of a 128-row unit land side by side; a 256-row slab is two units.
                // On a pair both CTAs' boxes of a hand-over are credited to the leader's barrier.
                Ring ra;
                for (int tile = first_tile; ok && tile < total_tiles; tile += tile_step) {
                    int mt, nt;
                    tile_coords<C::BAND>(tile, p.m_tiles, p.n_tiles, mt, nt);
                    const int row0 = mt * C::T_MC + row_off;
                    for (int k = 0; ok && k < p.k_steps; ++k) {
                        for (int h = 0; h < C::HA; ++h) {            // hand-overs of this K-step
                            if (!(ok = wait_bar_t<true, PAIR>(cx, a_empty + 8 * ra.stage, ra.phase ^ 1u, 0x002))) break;
                            const uint32_t dst = a_base + ra.stage * C::GPS * C::UNIT_BYTES;
                            if constexpr (PAIR) {
                                if (leader) mbar_arrive_expect_tx(a_full + 8 * ra.stage, 2 * C::GPS * C::UNIT_BYTES);
                                const uint32_t fa = mapa_shared(a_full + 8 * ra.stage, 0);
#pragma unroll
                                for (int sl = 0; sl < C::SPG; ++sl)
                                    tma_load_2d_pair(dst + sl * C::SLAB_BF16_BYTES, &tm_a, k * C::T_K, row0 + h * C::GPS * 128 + sl * T_MA, fa);
                            } else {
                                const uint32_t fa = a_full + 8 * ra.stage;
                                mbar_arrive_expect_tx(fa, C::GPS * C::UNIT_BYTES);
#pragma unroll
                                for (int sl = 0; sl < C::SPG; ++sl)
                                    tma_load_2d(dst + sl * C::SLAB_BF16_BYTES, &tm_a, k * C::T_K, row0 + h * C::GPS * 128 + sl * T_MA, fa);
                            }
                            ra.advance(C::NAH);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ================================ UMMA issuer (the leader's, on a pair) ========
        if (leader && elect_one()) {
            constexpr uint32_t idesc = umma_idesc_bf16_f32(PAIR ? 256 : 128, 256, false, false);   // both operands K-major
            Cursor<C::NAH, C::LAH> ra;               // hand-overs of A: one per 128-row unit, or per 256-row slab
            Cursor<C::NB, C::LB> rb;                 // first unit of this CTA's part of the B tile; a second follows it
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = first_tile; ok && tile < total_tiles; tile += tile_step, acc_phase ^= 1u) {
                for (int k = 0; ok && k < p.k_steps; ++k) {
                    // the converted B tile of this K-step: UB units per CTA, adjacent in shared memory
#pragma unroll
                    for (int u = 0; u < C::UB; ++u)
                        ok = ok && wait_bar_t<true, PAIR>(cx, b_full + 8 * (rb.bar + u), rb.phase, 0x101);
                    if (!ok) break;
                    const uint32_t bs = b_base + rb.buf() * C::UNIT_BYTES;
                    for (int g = 0; g < 2; ++g) {
                        if (k == 0 && !(ok = wait_bar_t<true, PAIR>(cx, acc_empty + 8 * g, acc_phase ^ 1u, 0x102))) break;
                        if ((g % C::GPS) == 0 && !(ok = wait_bar_t<true, PAIR>(cx, a_full + 8 * ra.bar, ra.phase, 0x103))) break;
                        tcgen05_fence_after_sync();
                        const uint32_t as = a_base + (ra.buf() * C::GPS + (g % C::GPS)) * C::UNIT_BYTES;
#pragma unroll
                        for (int kk = 0; kk < C::T_K / 16; ++kk) {
                            const uint64_t a_desc = umma_smem_desc_sw128(as + kk * 32, 16, 1024);
                            const uint64_t b_desc = umma_smem_desc_sw128(bs + kk * 32, 16, 1024);
                            if constexpr (PAIR)
                                umma_f16_ss_pair(tmem_base + static_cast<uint32_t>(g * 256), a_desc, b_desc, idesc, (k > 0 || kk > 0) ? 1u : 0u);
                            else
                                umma_f16_ss(tmem_base + static_cast<uint32_t>(g * 256), a_desc, b_desc, idesc, (k > 0 || kk > 0) ? 1u : 0u);
                        }
                        if ((g % C::GPS) == C::GPS - 1) {
                            cfg_commit<PAIR>(a_empty + 8 * ra.bar);
                            ra.template advance<1>();
                        }
                        if (k == p.k_steps - 1) cfg_commit<PAIR>(acc_full + 8 * g);
                    }
                    if (!ok) break;
#pragma unroll
                    for (int u = 0; u < C::UB; ++u) cfg_commit<PAIR>(b_empty + 8 * (rb.bar + u));
                    rb.template advance<C::UB>();
                }
            }
        }
    } else if (warp < kFirstDequantWarp) {
        // ================================ epilogue ====================================
        const int q = warp & 3;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = first_tile; ok && tile < total_tiles; tile += tile_step, acc_phase ^= 1u) {
            int mt, nt;
            tile_coords<C::BAND>(tile, p.m_tiles, p.n_tiles, mt, nt);
            for (int g = 0; g < 2; ++g) {
                if (!(ok = wait_bar_t<false, PAIR>(cx, acc_full + 8 * g, acc_phase, 0x201))) break;
                tcgen05_fence_after_sync();
                const int row0 = mt * C::T_MC + row_off + g * 128 + q * 32;
                const int col0 = nt * C::T_N;
                const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(g * 256);
                const uint32_t box = smem_base + stage_off + static_cast<uint32_t>(warp - kFirstEpilogueWarp) * kEpilogueBoxBytes;
                if (C_Q) epilogue_bfp16<C::T_N>(&tm_c, t_addr, box, lane, row0, col0, p.M, p.N, p.C_exp, p.c_exp_rows);
                else epilogue_bf16<C::T_N>(&tm_c, p.C, p.ldc, t_addr, box, lane, row0, col0, p.M, p.N);
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (PAIR) mbar_arrive_cluster(mapa_shared(acc_empty + 8 * g, 0));
                    else mbar_arrive(acc_empty + 8 * g);
                }
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    } else {
        // ================================ dequantisers ================================
        // The conversion jobs of this CTA in the order the UMMA issuer asks for their results: per K-step the UB
        // units of B (the issuer waits for the B tile first), then the JA hand-overs of A (config 2).  Group g
        // takes jobs g, g + 4, g + 8, ...; the rings' barrier counts (stream_bars) make every barrier the business
        // of one group.
        const int group = (threadIdx.x - kFirstDequantWarp * 32) / 128, t = (threadIdx.x - kFirstDequantWarp * 32) % 128;
        int64_t k_steps_total = 0;                    // K-steps over this CTA's tiles
        for (int tile = first_tile; tile < total_tiles; tile += tile_step) k_steps_total += p.k_steps;
        const int64_t jobs = k_steps_total * C::IPK;
        for (int64_t n = group; n < jobs; n += kCfgGroups) {
            const int64_t ks = n / C::IPK;
            const int j = static_cast<int>(n - ks * C::IPK);
            bool ok = true;
            if (A_Q && j >= C::UB) {
                if constexpr (A_Q)
                    ok = dequant_job<T_MA, C::NAS, C::LAR, C::NAH, C::LAH, PAIR>(cx, ks * C::HA + (j - C::UB), t, lane, ar_full, ar_empty, a_full,
                                                                                 a_empty, a_raw_base, a_base, 0x300);
            } else {
                ok = dequant_job<128, C::NBR, C::LBR, C::NB, C::LB, PAIR>(cx, ks * C::UB + j, t, lane, br_full, br_empty, b_full, b_empty,
                                                                          b_raw_base, b_base, 0x310);
            }
            if (!ok) break;
        }
    }

    // ---- teardown: on the abort path give copies and MMAs in flight time to land first; on a pair the
    // peer may still arrive on this CTA's barriers until it gets here ----
    if (*cx.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after_sync();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, 512u);
        else tmem_dealloc(tmem_base, 512u);
    }
}

std::mutex g_cfg_mutex;
unsigned int* g_cfg_flag_addr[64] = {};

template <int T_MA, bool A_Q, bool C_Q, bool PAIR>
atb_status_t launch_cfg(int64_t M, int64_t N, int64_t K, const void* A, const uint8_t* A_exp, int64_t lda,
                        const int8_t* Bt_mant, const uint8_t* Bt_exp, void* Cout, uint8_t* C_exp, int64_t ldc,
                        int num_sms, unsigned int* error_flag, cudaStream_t stream) {
    using C = CfgK<T_MA, A_Q, PAIR>;
    CUtensorMap tm_a, tm_a_exp, tm_b, tm_b_exp, tm_c;
    const int64_t M_pad = atb::round_up(M, 32), N_pad = atb::round_up(N, 32);
    if (A_Q) {
        if (!make_map_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, A, K, M, K, 64, T_MA, CU_TENSOR_MAP_SWIZZLE_NONE) ||
            !make_map_2d(&tm_a_exp, CU_TENSOR_MAP_DATA_TYPE_UINT64, 8, A_exp, M_pad, atb::ceil_div(K, 64), M_pad * 8, T_MA, 1,
                         CU_TENSOR_MAP_SWIZZLE_NONE))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the planes of A");
    } else {
        if (!make_map_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, K, M, lda * 2, 64, T_MA, CU_TENSOR_MAP_SWIZZLE_128B))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for A");
        tm_a_exp = tm_a;                                   // unused
    }
    if (!make_map_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Bt_mant, K, N, K, 64, 128, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&tm_b_exp, CU_TENSOR_MAP_DATA_TYPE_UINT64, 8, Bt_exp, N_pad, atb::ceil_div(K, 64), N_pad * 8, 128, 1,
                     CU_TENSOR_MAP_SWIZZLE_NONE))
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the planes of B");
    if (C_Q) {
        if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Cout, N, M, N, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B))
            return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the mantissa plane of C");
    } else if (!make_map_2d(&tm_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Cout, N, M, ldc * 2, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) {
        return atb::fail(ATB_ERR_CUDA, "cuTensorMapEncodeTiled failed for C");
    }
    CfgParams p;
    p.M = M; p.N = N; p.K = K; p.ldc = ldc;
    p.C = static_cast<__nv_bfloat16*>(Cout);
    p.m_tiles = static_cast<int>(atb::ceil_div(M, C::T_MC));
    p.n_tiles = static_cast<int>(atb::ceil_div(N, C::T_N));
    p.k_steps = static_cast<int>(atb::ceil_div(K, C::T_K));
    p.C_exp = C_exp;
    p.c_exp_rows = M_pad;
    p.error_flag = error_flag;
    auto kernel = atb_gemm_cfg_kernel<T_MA, A_Q, C_Q, PAIR>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(C::SMEM_BYTES));
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int units = PAIR ? num_sms / 2 : num_sms;      // CTAs, or CTA pairs
    const int n_units = static_cast<int>(tiles < units ? tiles : units);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(PAIR ? 2 * n_units : n_units), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, tm_a, tm_a_exp, tm_b, tm_b_exp, tm_c, p);
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "gemm (config) launch: %s", cudaGetErrorString(e));
    return ATB_OK;
}

}  // namespace

extern "C" atb_status_t atb_gemm_config_tiled(int config, int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                              const void* A_dev, const uint8_t* A_exp_dev, int64_t lda,
                                              const int8_t* Bt_mant_dev, const uint8_t* Bt_exp_dev,
                                              void* C_dev, uint8_t* C_exp_dev, int64_t ldc, void* stream) {
    atb::clear_error();
    if (config != 1 && config != 2) return atb::fail(ATB_ERR_BAD_TILING, "config=%d: 1 (A BF16, B BFP16, C BF16) or 2 (all BFP16)", config);
    if ((T_MC != 256 && T_MC != 512) || T_K != 64 || T_N != 256 || !(T_MA == 32 || T_MA == 64 || T_MA == 128 || T_MA == 256))
        return atb::fail(ATB_ERR_BAD_TILING, "the precision configurations run T_MC = 256 (one CTA) or 512 (a CTA pair), T_K = 64, T_N = 256 "
                                             "with T_MA in {32, 64, 128, 256} (got T_MA=%d, T_MC=%d, T_K=%d, T_N=%d)", T_MA, T_MC, T_K, T_N);
    if (!A_dev || !Bt_mant_dev || !Bt_exp_dev || !C_dev || (config == 2 && (!A_exp_dev || !C_exp_dev)))
        return atb::fail(ATB_ERR_NULL_POINTER, "operand pointers must be non-NULL");
    if (M < 1 || N < 16 || N % 16 != 0 || K < 16 || K % 16 != 0 || M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30))
        return atb::fail(ATB_ERR_BAD_SHAPE, "need M >= 1, N %% 16 == 0, K %% 16 == 0 (got %lld, %lld, %lld)", (long long)M, (long long)N, (long long)K);
    if (config == 1 && (lda < K || lda % 8 != 0 || ldc < N || ldc % 8 != 0))
        return atb::fail(ATB_ERR_BAD_SHAPE, "lda=%lld must be >= K, ldc=%lld >= N, both multiples of 8", (long long)lda, (long long)ldc);
    if (!atb::aligned16(A_dev) || !atb::aligned16(Bt_mant_dev) || !atb::aligned16(Bt_exp_dev) || !atb::aligned16(C_dev) ||
        (config == 2 && (!atb::aligned16(A_exp_dev) || !atb::aligned16(C_exp_dev))))
        return atb::fail(ATB_ERR_MISALIGNED, "all device pointers must be 16-byte aligned");
    int dev = 0, major = 0, minor = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (major != 10 || minor != 0)
        return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d; this library runs on 10.0 only", major, minor);
    if (dev < 0 || dev >= 64) return atb::fail(ATB_ERR_UNSUPPORTED_DEVICE, "device ordinal %d out of range", dev);
    unsigned int* flag = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_cfg_mutex);
        if (!g_cfg_flag_addr[dev]) {
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&g_cfg_flag_addr[dev]), g_cfg_error_flag);
            if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        }
        flag = g_cfg_flag_addr[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define ATB_CFG_CASE(TMA_, PAIR_)                                                                                              \
    if (T_MA == TMA_ && (T_MC == 512) == PAIR_) {                                                                              \
        if (config == 1)                                                                                                       \
            return launch_cfg<TMA_, false, false, PAIR_>(M, N, K, A_dev, nullptr, lda, Bt_mant_dev, Bt_exp_dev, C_dev, nullptr, ldc, sms, flag, st); \
        return launch_cfg<TMA_, true, true, PAIR_>(M, N, K, A_dev, A_exp_dev, K, Bt_mant_dev, Bt_exp_dev, C_dev, C_exp_dev, N, sms, flag, st);      \
    }
    ATB_CFG_CASE(32, false) ATB_CFG_CASE(64, false) ATB_CFG_CASE(128, false) ATB_CFG_CASE(256, false)
    ATB_CFG_CASE(32, true) ATB_CFG_CASE(64, true) ATB_CFG_CASE(128, true) ATB_CFG_CASE(256, true)
#undef ATB_CFG_CASE
    return atb::fail(ATB_ERR_BAD_TILING, "no kernel for T_MA=%d, T_MC=%d", T_MA, T_MC);
}

extern "C" atb_status_t atb_gemm_config(int config, int64_t M, int64_t N, int64_t K,
                                        const void* A_dev, const uint8_t* A_exp_dev, int64_t lda,
                                        const int8_t* Bt_mant_dev, const uint8_t* Bt_exp_dev,
                                        void* C_dev, uint8_t* C_exp_dev, int64_t ldc, void* stream) {
    // the CTA pair shares the converted B tile between two SMs; a problem of one 256-row tile has no use for it
    return atb_gemm_config_tiled(config, M, N, K, 128, M > 256 ? 512 : 256, 64, 256, A_dev, A_exp_dev, lda, Bt_mant_dev, Bt_exp_dev, C_dev,
                                 C_exp_dev, ldc, stream);
}

namespace atb {
// Reads and clears the timeout flag of the configuration kernels (part of atb_device_status).
unsigned int take_cfg_error_flag() {
    unsigned int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_cfg_error_flag, sizeof flag) != cudaSuccess) return 0;
    if (flag != 0) {
        const unsigned int zero = 0;
        cudaMemcpyToSymbol(g_cfg_error_flag, &zero, sizeof zero);
    }
    return flag;
}
}  // namespace atb

#ifdef ATB_PROFILE
// Diagnostic build only: wait-cycle counters of the configuration kernels (16 values), read and cleared.
extern "C" int atb_debug_read_wait_cycles_cfg(unsigned long long* out16) { return read_wait_cycles(out16); }
#endif
