// Device-side building blocks shared by the GEMM kernels (single-CTA and CTA-pair): bounded
// mbarrier waits, ring bookkeeping, tile rasterisation, the BFP16 -> BF16 dequantiser, and the
// host helper that encodes TMA descriptors.  Everything lives in an unnamed namespace: each
// translation unit gets its own copy.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "atb_internal.h"
#include "bfp16_block.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kKA = 64;               // columns of A per raw slab and per converted operand group, whatever T_K is
constexpr int kDequantWarps = 16;
constexpr int kThreads = (7 + kDequantWarps) * 32;      // + B producer, UMMA issuer, 4 epilogue warps, A producer
constexpr int kAProducerWarp = 6 + kDequantWarps;       // the last warp
// The dequantiser warps work in groups; slabs are dealt to the groups in turn, so that several
// slabs are in flight and every thread has a few 16-element slots per barrier round trip.
// An mbarrier wait only tells two consecutive phases apart, so every barrier must see its phases
// completed and awaited strictly in order by ONE group.  A ring of n buffers served by d groups
// therefore has lcm(n, d) barrier pairs: slab c lives in buffer c mod n and is guarded by barrier
// c mod lcm(n, d), which is always the business of group c mod d.  Ring depths are then free of
// the group count.
__host__ __device__ constexpr int dq_groups(int T_MA, int T_K, int T_N) {
#ifdef ATB_DQ_GROUPS
    return ATB_DQ_GROUPS;
#else
    // two groups for 256-row slabs, and where a double-buffered B tile already takes 128 KB
    return (T_MA >= 256 || T_K * T_N >= 128 * 256) ? 2 : 4;
#endif
}
constexpr int kFirstEpilogueWarp = 2;
constexpr int kFirstDequantWarp = 6;
constexpr int kMaxStages = 16;
constexpr int kMaxRingBars = 32;
constexpr uint32_t kEpilogueBoxBytes = 32 * 128;   // 32 rows x 64 bf16 columns
// The CTA-pair kernel stages C in full-size boxes (128-byte rows) where 64- and 128-row slabs leave room
// for them, and in half-size boxes under 32-row slabs, whose deeper raw ring needs the space.
constexpr int pair_box_cols(int slab, int T_N = 512) { return (slab >= 64 || T_N == 256) ? 64 : 32; }
constexpr uint32_t pair_box_bytes(int slab, int T_N = 512) { return 32u * pair_box_cols(slab, T_N) * 2u; }
constexpr uint32_t kSmemBudget = 232448;          // 227 KB of dynamic shared memory per CTA
#ifdef ATB_TEST_WAIT_NS                             // test build of the timeout path only: a short limit
constexpr uint64_t kWaitTimeoutNs = ATB_TEST_WAIT_NS;
#else
constexpr uint64_t kWaitTimeoutNs = 2000000000ull;  // every mbarrier wait gives up after 2 s
#endif

// lcm(n, d) for d a power of two: the number of barrier pairs of a ring of n buffers and d groups
__host__ __device__ constexpr int ring_bars(int n, int d) {
    int g = d;
    while (n % g) g >>= 1;
    return n / g * d;
}

using atb::slab_bundle;

// ---------------------------------------------------------------------------------------------
// Ring plans: how the 227 KB of shared memory are split between the B ring, the raw-slab ring and
// the ring of dequantised 128-row groups.  Evaluated at compile time (the kernels take the depths
// as constants) and at run time (atb_tiling_plan, the tiling selection) from the same functions.
// ---------------------------------------------------------------------------------------------
struct RingPlan {
    bool ok = false;
    int nb = 2, ng = 2, nr = 1;      // B stages, dequantised 128-row groups, raw slabs
    int dqg = 1;                     // dequantiser groups
    int acc_bufs = 1, tmem_cols = 32;
    uint32_t smem_bytes = 0;
};

constexpr uint32_t ring_smem_bytes(uint32_t b_bytes, uint32_t group_bytes, uint32_t raw_bytes, int acc_bars,
                                   int dqg, int bundle, int b, int g, int n_deq, int r, uint32_t box_bytes = kEpilogueBoxBytes) {
    const uint32_t bars = 8u * (2 * b + 2 * ring_bars(r, dqg * bundle) + 2 * ring_bars(n_deq, dqg) + 2 * acc_bars) + 16u;
    return 1024u + b * b_bytes + g * group_bytes + r * raw_bytes + 1024u + 4u * box_bytes + bars;
}

// Single-CTA kernel, tiling (T_MA, T_MC, T_K, T_N).
constexpr RingPlan plan_single(int T_MA, int T_MC, int T_K, int T_N) {
    RingPlan pl;
    if (!(T_MC == 128 || T_MC == 256 || T_MC == 384)) return pl;
    if (!(T_N == 64 || T_N == 128 || T_N == 256 || T_N == 512)) return pl;
    if (!(T_K == 64 || T_K == 128)) return pl;
    if (!(T_MA == 32 || T_MA == 64 || T_MA == 128 || T_MA == 256) || T_MA > T_MC || T_MC % T_MA != 0) return pl;
    const int G = T_MC / 128;
    if (G * T_N > 512) return pl;
    const uint32_t b_bytes = T_K * T_N * 2, group_bytes = 128 * kKA * 2, raw_bytes = T_MA * kKA * 9 / 8;
    const int gps = T_MA > 128 ? T_MA / 128 : 1;          // groups per slab
    const int spg = T_MA < 128 ? 128 / T_MA : 1;          // slabs per group
    const int dqg = dq_groups(T_MA, T_K, T_N);
    pl.dqg = dqg;
    pl.acc_bufs = (2 * G * T_N <= 512) ? 2 : 1;
    int cols = 32;
    while (cols < pl.acc_bufs * G * T_N) cols <<= 1;
    pl.tmem_cols = cols;
    // dequantised stages of a plan with g groups; the UMMA issuer takes spg of them at a time
    const auto total = [=](int b, int g, int r) {
        return ring_smem_bytes(b_bytes, group_bytes, raw_bytes, 2 * G, dqg, slab_bundle(spg, r, dqg), b, g,
                               T_MA <= 128 ? g * (spg / slab_bundle(spg, r, dqg)) : g / gps, r);
    };
    const auto bars_ok = [=](int g, int r) {
        return ring_bars(r, dqg * slab_bundle(spg, r, dqg)) <= kMaxRingBars &&
               ring_bars(T_MA <= 128 ? g * (spg / slab_bundle(spg, r, dqg)) : g / gps, dqg) <= kMaxRingBars;
    };
    // Any depth is legal (see ring_bars); the default plan gives every dequantiser group the same
    // number of raw slabs and of dequantised stages, which measured best: one raw slab fewer than
    // groups costs 10 %, one more gains nothing.
    // Raw ring: whole rounds of the dequantiser groups over whole bundles (dqg * spg slabs) where that
    // fits; a tiling that only fits with fewer slabs gets one slab per group and smaller bundles.
    const int ng_step = T_MA <= 128 ? (dqg >= spg ? dqg / spg : 1) : dqg * gps;
    int nb = 2, ng = ng_step < 2 ? 2 * ng_step : ng_step;
    int nr_step = dqg * spg;                             // 512 rows x 64 columns of look-ahead
    if (total(nb, ng, nr_step) > kSmemBudget) nr_step = dqg;
    int nr = nr_step;
    pl.nb = nb; pl.ng = ng; pl.nr = nr;
    if (total(nb, ng, nr) > kSmemBudget) return pl;
    // Grow the rings towards a target look-ahead, counted in 128-row x T_K operand groups:
    // B tiles hide the TMA latency for G groups each, raw slabs for T_MA/128 groups each.
    const double target_b = 8.0 * 64 / T_K, target_r = 6.0, target_g = 4.0;
    for (;;) {
        const double cov_b = nb * G / target_b, cov_r = nr * (T_MA / 128.0) / target_r, cov_g = ng / target_g;
        int pick = -1;
        double best = 1.0;                               // stop once every ring meets its target
        if (cov_b < best && nb < kMaxStages && total(nb + 1, ng, nr) <= kSmemBudget) { best = cov_b; pick = 0; }
        if (cov_r < best && nr + nr_step <= kMaxStages && bars_ok(ng, nr + nr_step) && total(nb, ng, nr + nr_step) <= kSmemBudget) { best = cov_r; pick = 1; }
        if (cov_g < best && ng + ng_step <= kMaxStages && bars_ok(ng + ng_step, nr) && total(nb, ng + ng_step, nr) <= kSmemBudget) { best = cov_g; pick = 2; }
        if (pick < 0) break;
        if (pick == 0) ++nb; else if (pick == 1) nr += nr_step; else ng += ng_step;
    }
#if defined(ATB_RINGS_NB) && defined(ATB_RINGS_NG) && defined(ATB_RINGS_NR)
    // Tuning build: fixed depths wherever they are valid for the tiling and fit.
    if (ATB_RINGS_NB >= 2 && ATB_RINGS_NG >= gps && ATB_RINGS_NG % gps == 0 && ATB_RINGS_NR >= 1 &&
        bars_ok(ATB_RINGS_NG, ATB_RINGS_NR) && total(ATB_RINGS_NB, ATB_RINGS_NG, ATB_RINGS_NR) <= kSmemBudget) {
        nb = ATB_RINGS_NB; ng = ATB_RINGS_NG; nr = ATB_RINGS_NR;
    }
#endif
    pl.nb = nb; pl.ng = ng; pl.nr = nr;
    pl.smem_bytes = total(nb, ng, nr);
    pl.ok = true;
    return pl;
}

// CTA-pair kernel; `slab` = T_MA <= 128 rows.  Two forms:
//   T_N = 512, T_K = 64: one 256 x 512 tile per pair; each CTA holds a 128 x 512 accumulator (all of its tensor
//                        memory), one buffer.
//   T_N = 256, T_K = 128: two 128 x 256 tiles, one above the other, per pair (the tiling 128, 128, 256 on more than
//                        one tile row): each CTA holds its 128 x 256 accumulator twice, so the epilogue of a tile -
//                        bound by what one SM can store per unit of time - runs beside the K loop of the next
//                        tile.  A B stage is 128 rows deep: two 64-column rounds of A per stage keep the K-step
//                        at 1024 tensor cycles, the rate at which the leader needs both CTAs' operands.
constexpr RingPlan plan_pair(int slab, int T_N = 512) {
    RingPlan pl;
    if (!(slab == 32 || slab == 64 || slab == 128) || !(T_N == 512 || T_N == 256)) return pl;
    const int slabs = 128 / slab;
    const bool wide = T_N == 512;
    // this CTA's half of a B stage: 128 columns of every 256-column chunk, 64 (wide) or 128 rows deep: 32 KB either way
    const uint32_t b_bytes = 4 * 64 * 128, group_bytes = 128 * 64 * 2, raw_bytes = slab * 64 * 9 / 8;
    const int dqg = 4;
    pl.dqg = dqg;
    pl.acc_bufs = wide ? 1 : 2;
    pl.tmem_cols = 512;
    const auto total = [=](int b, int g, int r) {
        return ring_smem_bytes(b_bytes, group_bytes, raw_bytes, 2, dqg, slab_bundle(slabs, r, dqg), b, g,
                               g * (slabs / slab_bundle(slabs, r, dqg)), r, pair_box_bytes(slab, T_N));
    };
    const auto bars_ok = [=](int g, int r) {
        return ring_bars(r, dqg * slab_bundle(slabs, r, dqg)) <= kMaxRingBars &&
               ring_bars(g * (slabs / slab_bundle(slabs, r, dqg)), dqg) <= kMaxRingBars;
    };
    // as in plan_single: whole rounds of the dequantiser groups
    int ng = (dqg + slabs - 1) / slabs;
    if ((ng * slabs) % dqg != 0) ng = dqg;
    const int ng_step = ng;
    int nb = 3, nr = dqg;
    pl.nb = nb; pl.ng = ng; pl.nr = nr;
    if (total(nb, ng, nr) > kSmemBudget) return pl;
    // Spend what is left on bf16 groups, raw slabs (up to 8 K-steps of look-ahead), then B tiles
    // (measured: the dequantised-A ring is the one whose depth pays most).
    while (ng + ng_step <= 4 && bars_ok(ng + ng_step, nr) && total(nb, ng + ng_step, nr) <= kSmemBudget) ng += ng_step;
    while (nr + dqg <= kMaxStages && nr * slab < 8 * 128 && bars_ok(ng, nr + dqg) && total(nb, ng, nr + dqg) <= kSmemBudget) nr += dqg;
    // a fifth group where it still fits (under 32-row slabs, whose epilogue boxes are half-size): measured +3 % there
    if (ng == 4 && bars_ok(5, nr) && total(nb, 5, nr) <= kSmemBudget) ng = 5;
    while (nb < 4 && total(nb + 1, ng, nr) <= kSmemBudget) ++nb;
#if defined(ATB_RINGS_NB) && defined(ATB_RINGS_NG) && defined(ATB_RINGS_NR)
    if (ATB_RINGS_NB >= 2 && ATB_RINGS_NG >= 1 && ATB_RINGS_NR >= 1 && bars_ok(ATB_RINGS_NG, ATB_RINGS_NR) &&
        total(ATB_RINGS_NB, ATB_RINGS_NG, ATB_RINGS_NR) <= kSmemBudget) {
        nb = ATB_RINGS_NB; ng = ATB_RINGS_NG; nr = ATB_RINGS_NR;
    }
#endif
    pl.nb = nb; pl.ng = ng; pl.nr = nr;
    pl.smem_bytes = total(nb, ng, nr);
    pl.ok = true;
    return pl;
}

struct GemmParams {
    int64_t M, N, K, ldc;
    __nv_bfloat16* C;
    int m_tiles, n_tiles, k_steps;
    unsigned int* error_flag;
    uint8_t* C_exp;      // quantising epilogue: exponent plane of C [ceil(N/64)][c_exp_rows][8]
    int64_t c_exp_rows;  // roundup(M, 32)
    int splits;          // split-K: each output tile is computed as `splits` partial tiles over K ranges
    int m_pad;           // split-K: rows per split in the FP32 workspace (m_tiles * T_MC)
};

// One unit of work of a persistent CTA: an output tile and the K-steps [k_begin, k_end) of it.
struct WorkItem {
    int mt, nt, k_begin, k_end, split;
};

struct Ring {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int n) {
        if (++stage == n) { stage = 0; phase ^= 1u; }
    }
};

// Position of a slab in a ring of N buffers guarded by L = ring_bars(N, groups) barrier pairs.
// `phase` is the parity of the barrier phase that belongs to this slab.  All sizes are compile-time
// constants; with L == N the buffer index and the barrier index are one variable.
template <int N, int L>
struct Cursor {
    static_assert(L >= N && L % N == 0, "L is a multiple of N");
    int bar = 0, buf_ = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void start_at(int slab) {       // slab < L
        bar = slab;
        buf_ = slab % N;
    }
    __device__ __forceinline__ int buf() const { return L == N ? bar : buf_; }
    template <int STEP>
    __device__ __forceinline__ void advance() {
        static_assert(STEP <= L, "step");
        bar += STEP;
        if (bar >= L) { bar -= L; phase ^= 1u; }
        if (L != N) {
            buf_ += STEP % N;
            if (buf_ >= N) buf_ -= N;
        }
    }
    // Barrier index and parity of the slab N places back - the last user of this slab's buffer.
    // For the first N slabs that is a phase "before the first", which a fresh barrier reports
    // as complete.
    __device__ __forceinline__ int freed_bar() const { return (L == N || bar < N) ? bar - N + L : bar - N; }
    __device__ __forceinline__ uint32_t freed_parity() const { return (L == N || bar < N) ? phase ^ 1u : phase; }
};

struct Ctx {
    volatile uint32_t* abort_flag;
    unsigned int* error_flag;
};

// Bounded mbarrier wait.  Returns false when the CTA is aborting or the wait timed out.
// kSpin = true (single-thread, latency-critical roles: TMA producer, UMMA issuer): tight polling.
// kSpin = false (whole warps): after a first immediate probe the hardware may suspend the thread
// for up to `kSuspendNs` per probe, so that waiting warps do not take issue slots from the
// dequantisers.  kCluster = true uses cluster-scope acquire (arrivals may come from the peer CTA).
constexpr uint32_t kSuspendNs = 20000;
template <bool kSpin, bool kCluster>
__device__ __forceinline__ bool wait_bar_impl(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
    auto probe = [&]() { return kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    auto probe_suspend = [&]() {
        return kCluster ? mbar_try_wait_cluster_suspend(bar, parity, kSuspendNs) : mbar_try_wait_suspend(bar, parity, kSuspendNs);
    };
    if (probe()) return true;
    const uint64_t t0 = global_timer_ns();
    constexpr uint32_t kCheckMask = kSpin ? 1023u : 7u;
    for (uint32_t spins = 0;; ++spins) {
        if (kSpin ? probe() : probe_suspend()) return true;
        if ((spins & kCheckMask) == kCheckMask) {
            if (*cx.abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitTimeoutNs) {
                *cx.abort_flag = 1u;
                atomicCAS(cx.error_flag, 0u, code);
                return false;
            }
        }
    }
}
#ifdef ATB_PROFILE
// Opt-in diagnostic build (-DATB_PROFILE): cycles spent in each kind of wait, one row per CTA, one
// lane per warp reporting.  Slot = (role << 2 | barrier kind) taken from the wait's code.
__device__ unsigned long long g_wait_cycles[256][16];
// Host: sums the counters of this translation unit's kernels over the CTAs into out16, then clears them.
inline int read_wait_cycles(unsigned long long* out16) {
    static unsigned long long host[256][16];
    if (cudaDeviceSynchronize() != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(host, g_wait_cycles, sizeof host) != cudaSuccess) return 1;
    for (int j = 0; j < 16; ++j) { out16[j] = 0; for (int i = 0; i < 256; ++i) out16[j] += host[i][j]; }
    for (auto& row : host) for (auto& v : row) v = 0;
    return cudaMemcpyToSymbol(g_wait_cycles, host, sizeof host) == cudaSuccess ? 0 : 1;
}
#endif
template <bool kSpin, bool kCluster>
__device__ __forceinline__ bool wait_bar_t(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
#ifdef ATB_PROFILE
    const long long t0 = clock64();
    const bool ok = wait_bar_impl<kSpin, kCluster>(cx, bar, parity, code);
    if ((threadIdx.x & 31) == 0 || kSpin)
        atomicAdd(&g_wait_cycles[blockIdx.x & 255][((code >> 8) << 2 | (code & 3)) & 15],
                  static_cast<unsigned long long>(clock64() - t0));
    return ok;
#else
    return wait_bar_impl<kSpin, kCluster>(cx, bar, parity, code);
#endif
}
__device__ __forceinline__ bool wait_bar(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
    return wait_bar_t<false, false>(cx, bar, parity, code);
}
__device__ __forceinline__ bool wait_bar_spin(const Ctx& cx, uint32_t bar, uint32_t parity, unsigned code) {
    return wait_bar_t<true, false>(cx, bar, parity, code);
}

// BAND tile-rows per band: the CTAs of a wave (148 tiles, or 74 pair tiles) cover BAND row panels of the
// operand on the M side and 148 / BAND column panels of the other; the bytes a wave pulls through the L2 are
// least where the two sides weigh the same, BAND^2 = units * (bytes of a column panel) / (bytes of a row panel).
// atb_gemm (BFP16 row panels of 256 rows against BF16 column panels of 256 or 512 columns): 16.
template <int BAND = 16>
__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int& mt, int& nt) {
    // Bands of BAND tile-rows, column-major inside a band: the CTAs of one wave share a few
    // A row-panels and B column-panels in L2.
    const int per_band = BAND * n_tiles;
    const int band = tile / per_band, i = tile - band * per_band;
    const int rows = min(BAND, m_tiles - band * BAND);
    mt = band * BAND + i % rows;
    nt = i / rows;
    // odd bands walk the columns backwards: they start on the B panels the band before them ended on
    if (band & 1) nt = n_tiles - 1 - nt;
}

// K-step that a CTA loads `k0` steps into its `it`-th work item over [k_begin, k_end): every other work
// item of a CTA walks K downwards.  The CTAs of a wave move through K together and the next wave re-reads
// the same band of A panels; walking back, it starts on the K range that was touched last and still sits
// in the L2, where a second upward walk would find the least recently used - evicted - end first.
// Measured at 8192^3: 19 % fewer DRAM reads (CTA pair 583 -> 473 MB, single CTA 550 -> 447 MB), +0.7 % rate
// timed alone and +1.4 % under the power cap.  The price: the order of a tile's FP32 additions depends on
// its place in the walk.  That place is the same for every T_MA of a (T_MC, T_K, T_N) - C stays bit-identical
// across slab heights - but tilings of different tile shape, and the single-CTA and CTA-pair kernels, agree
// bit for bit only where no CTA computes more than one tile.  -DATB_FORWARD_K builds the upward-only walk.
__device__ __forceinline__ int serpentine_k(int it, int k0, int k_begin, int k_end) {
#ifndef ATB_FORWARD_K
    return (it & 1) ? k_begin + k_end - 1 - k0 : k0;
#else
    (void)it; (void)k_begin; (void)k_end;
    return k0;
#endif
}

template <bool SPLIT>
__device__ __forceinline__ WorkItem work_item(int item, const GemmParams& p) {
    WorkItem w;
    if (SPLIT) {
        const int total_tiles = p.m_tiles * p.n_tiles;
        w.split = item / total_tiles;
        tile_coords(item - w.split * total_tiles, p.m_tiles, p.n_tiles, w.mt, w.nt);
        w.k_begin = static_cast<int>(static_cast<int64_t>(w.split) * p.k_steps / p.splits);
        w.k_end = static_cast<int>(static_cast<int64_t>(w.split + 1) * p.k_steps / p.splits);
    } else {
        w.split = 0;
        tile_coords(item, p.m_tiles, p.n_tiles, w.mt, w.nt);
        w.k_begin = 0;
        w.k_end = p.k_steps;
    }
    return w;
}

// ---------------------------------------------------------------------------------------------
// Dequantise one raw slab (T_MA rows x T_K columns) into its place in a bf16 operand group.
// One group of dequantiser warps (GROUP_THREADS threads) works on a slab.  Thread t owns slot (row r, pair p) = (t / SPR + i *
// GROUP_THREADS / SPR, t % SPR), a slot being two blocks: 16 mantissa bytes (one 16-byte load; the loads of
// a warp are contiguous), two exponent bytes, and two 16-byte stores into the swizzled row.
//
// Per pair of elements (all packed, two values per 32-bit register):
//   1. prmt drops the bytes u = m + 128 (1..255) into the mantissas of two fp16 values 1024
//      (0x64uu = 1024 + u); subtracting 1024 (add.f16x2) normalises them: u as fp16, exact.
//   2. u is positive and non-zero, so fp16 -> bf16 is pure bit arithmetic: drop 3 mantissa bits
//      (they are zero: u has at most 8 significant bits) and re-bias the exponent by 112 -
//      (h >> 3) + 0x3800 per half, done for both halves by one mad.hi.u32 (x * 2^29 >> 32).  Re-biasing
//      by 6 more gives u / 64 instead of u.
//   3. one fma.rn.bf16x2 forms (u / 64) * s' - 2 s' = m * 2^(E-133) with s' = 2^(E-127): both products are
//      exact and so is the result (7 significant bits), bf16-subnormal results included (no flush to zero).
// The scales need no table: the exponent byte of a block IS the UE8M0 number 2^(E-127), so one
// cvt.rn.bf16x2.ue8m0x2 turns the two exponent bytes of a slot into the two scales s', a prmt each copies
// them into both halves, and -2 s' is one bf16x2 multiplication (exact, subnormal s' for E = 0 included).
// (An earlier version read s = 2^(E-133) and -128 s from a 256-entry table in shared memory: two 8-byte
// loads per slot, a quarter of the dequantisers' shared-memory wavefronts; without them the single-CTA
// tilings gained 1-3 %.)
// -2 s' is not a bf16 number for E >= 254: a thread that met such a block converts its slots of the slab
// once more in the two-step form, add.bf16x2 (u - 128, exact) then mul.bf16x2 by s = 2^(E-133).
// Only the prmt runs on the integer ALU pipe; the other operations go to the FMA pipe.
template <uint32_t kRebias>
__device__ __forceinline__ uint32_t bf16x2_of_bytes(uint32_t u, uint32_t selector) {
    const uint32_t h2 = __byte_perm(u, 0x64646464u, selector);
    uint32_t t, b;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(t) : "r"(h2), "r"(0xE400E400u));          // - 1024
    asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(b) : "r"(t), "r"(0x20000000u), "r"(kRebias));
    return b;
}
__device__ __forceinline__ uint32_t dequant_pair(uint32_t u, uint32_t selector, uint32_t scale2, uint32_t offset2) {
    uint32_t r;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(bf16x2_of_bytes<0x35003500u>(u, selector)), "r"(scale2), "r"(offset2));
    return r;
}
__device__ __forceinline__ uint32_t dequant_pair_two_step(uint32_t u, uint32_t selector, uint32_t scale2) {
    uint32_t d, r;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(bf16x2_of_bytes<0x38003800u>(u, selector)), "r"(0xC300C300u));   // - 128
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(d), "r"(scale2));
    return r;
}
// s = 2^(E-133) as bf16 in both halves of a word (bf16-subnormal for E < 7).  (E = 255, which the quantiser
// never writes, gives m * 2^122 like any other block - +-Inf beyond bf16.)
__device__ __forceinline__ uint32_t scale_bits(uint32_t E) {
    return ((E >= 7u) ? ((E - 6u) << 7) : (1u << E)) * 0x10001u;
}

// N slots of one thread: 16 mantissa bytes each (w, two's complement) of two blocks with exponents
// (e & 0xFF, e >> 8) -> two 16-byte stores of bf16 values per slot (addresses st0[i], st1[i]).
// FAST: the one-fma form; returns a word whose bit 31 is clear when a block had E >= 254 - the caller then
// converts again in the two-step form (FAST = false) before it hands the operand on.  The test stays off
// the conversion's dependency chain that way.
template <int N, bool FAST>
__device__ __forceinline__ uint32_t dequant_slots(const uint4 (&w)[N], const uint32_t (&e)[N],
                                                  const uint32_t (&st0)[N], const uint32_t (&st1)[N]) {
    uint32_t mx = 0u;                            // largest 2^(E-127) met, per half
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const uint32_t u0 = w[i].x ^ 0x80808080u, u1 = w[i].y ^ 0x80808080u;
        const uint32_t u2 = w[i].z ^ 0x80808080u, u3 = w[i].w ^ 0x80808080u;
        if constexpr (FAST) {
            uint32_t sp, c0, c1;
            asm("cvt.rn.bf16x2.ue8m0x2 %0, %1;" : "=r"(sp) : "h"(static_cast<uint16_t>(e[i])));
            asm("max.u16x2 %0, %1, %2;" : "=r"(mx) : "r"(mx), "r"(sp));
            const uint32_t s0 = __byte_perm(sp, 0, 0x1010), s1 = __byte_perm(sp, 0, 0x3232);
            asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(c0) : "r"(s0), "r"(0xC000C000u));       // -2 s'
            asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(c1) : "r"(s1), "r"(0xC000C000u));
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(st0[i]),
                         "r"(dequant_pair(u0, 0x4140u, s0, c0)), "r"(dequant_pair(u0, 0x4342u, s0, c0)),
                         "r"(dequant_pair(u1, 0x4140u, s0, c0)), "r"(dequant_pair(u1, 0x4342u, s0, c0))
                         : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(st1[i]),
                         "r"(dequant_pair(u2, 0x4140u, s1, c1)), "r"(dequant_pair(u2, 0x4342u, s1, c1)),
                         "r"(dequant_pair(u3, 0x4140u, s1, c1)), "r"(dequant_pair(u3, 0x4342u, s1, c1))
                         : "memory");
        } else {
            const uint32_t s0 = scale_bits(e[i] & 0xFFu), s1 = scale_bits(e[i] >> 8);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(st0[i]),
                         "r"(dequant_pair_two_step(u0, 0x4140u, s0)), "r"(dequant_pair_two_step(u0, 0x4342u, s0)),
                         "r"(dequant_pair_two_step(u1, 0x4140u, s0)), "r"(dequant_pair_two_step(u1, 0x4342u, s0))
                         : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(st1[i]),
                         "r"(dequant_pair_two_step(u2, 0x4140u, s1)), "r"(dequant_pair_two_step(u2, 0x4342u, s1)),
                         "r"(dequant_pair_two_step(u3, 0x4140u, s1)), "r"(dequant_pair_two_step(u3, 0x4342u, s1))
                         : "memory");
        }
    }
    // a block with E >= 254 has s' >= 2^127 = 0x7F00 as bf16, whose double is not a bf16 number
    return ((mx + 0x01000100u) & 0x80008000u) ? 0u : 0xFFFFFFFFu;
}

// Per-thread constants of the dequantiser: thread t of a group owns slot t (16 mantissas = blocks
// 2p, 2p+1 of row r0) of every ROWS_PER_ITER-row band of a slab.  All shared-memory offsets of the
// thread are fixed; a slab only moves the base addresses.
template <class C>
struct DequantLane {
    uint32_t ld_off, exp_off, st_off0, st_off1;
    __device__ __forceinline__ DequantLane(int t, int slab_rows) {
        const int p = t % C::SLOTS_PER_ROW, r0 = t / C::SLOTS_PER_ROW, kb = 2 * p;
        const uint32_t sw = static_cast<uint32_t>(r0 & 7);                  // ROWS_PER_ITER is a multiple of 8
        ld_off = static_cast<uint32_t>(t) * 16u;
        exp_off = static_cast<uint32_t>((kb >> 3) * slab_rows * 8 + r0 * 8 + (kb & 7));
        const uint32_t row = static_cast<uint32_t>((kb >> 3)) * C::KHALF_BYTES + static_cast<uint32_t>(r0) * 128u;
        st_off0 = row + (((static_cast<uint32_t>(kb) & 7u) ^ sw) << 4);
        st_off1 = row + ((((static_cast<uint32_t>(kb) & 7u) + 1u) ^ sw) << 4);
    }
};

// Dequantises one slab: raw mantissas / exponents in shared memory -> bf16 operand rows starting at
// row `row_base` (a multiple of 32) of the 128-row groups at dst_base.
template <class C, bool FAST = true>
__device__ __forceinline__ void dequant_slab(const DequantLane<C>& ln, uint32_t raw_mant, uint32_t raw_exp,
                                             uint32_t dst_base, int row_base, int t, int T_MA_rows) {
    static_assert(C::ROWS_PER_ITER % 8 == 0 && 128 % C::ROWS_PER_ITER == 0, "band height");
    const uint32_t ld = raw_mant + ln.ld_off, le = raw_exp + ln.exp_off;
    const uint32_t st0 = dst_base + static_cast<uint32_t>(row_base) * 128u + ln.st_off0;
    const uint32_t st1 = dst_base + static_cast<uint32_t>(row_base) * 128u + ln.st_off1;
    const int r0 = t / C::SLOTS_PER_ROW;
    uint4 w[C::DQ_ITERS];
    uint32_t e[C::DQ_ITERS];
#pragma unroll
    for (int i = 0; i < C::DQ_ITERS; ++i) {
        if (C::SLOTS % C::GROUP_THREADS == 0 || r0 + i * C::ROWS_PER_ITER < T_MA_rows) {
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[i].x), "=r"(w[i].y), "=r"(w[i].z), "=r"(w[i].w)
                         : "r"(ld + static_cast<uint32_t>(i * C::GROUP_THREADS * 16)));
            uint16_t e2;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(e2) : "r"(le + static_cast<uint32_t>(i * C::ROWS_PER_ITER * 8)));
            e[i] = e2;
        }
    }
    // band i starts i * ROWS_PER_ITER rows further on: possibly in the next 128-row group
    constexpr uint32_t kBandRows = C::ROWS_PER_ITER;
    uint32_t all = 0xFFFFFFFFu;
    if constexpr (C::SLOTS % C::GROUP_THREADS == 0) {
        constexpr int CHUNK = C::DQ_ITERS < 4 ? C::DQ_ITERS : 4;             // slots converted under one test
        static_assert(C::DQ_ITERS % CHUNK == 0, "whole chunks");
#pragma unroll
        for (int i0 = 0; i0 < C::DQ_ITERS; i0 += CHUNK) {
            uint4 wc[CHUNK];
            uint32_t ec[CHUNK], a0[CHUNK], a1[CHUNK];
#pragma unroll
            for (int j = 0; j < CHUNK; ++j) {
                const int i = i0 + j;
                const uint32_t band = static_cast<uint32_t>((i * kBandRows) >> 7) * C::GROUP_BYTES + static_cast<uint32_t>((i * kBandRows) & 127) * 128u;
                wc[j] = w[i]; ec[j] = e[i]; a0[j] = st0 + band; a1[j] = st1 + band;
            }
            all &= dequant_slots<CHUNK, FAST>(wc, ec, a0, a1);
        }
    } else {
#pragma unroll
        for (int i = 0; i < C::DQ_ITERS; ++i) {
            if (r0 + i * C::ROWS_PER_ITER < T_MA_rows) {
                const uint32_t band = static_cast<uint32_t>((i * kBandRows) >> 7) * C::GROUP_BYTES + static_cast<uint32_t>((i * kBandRows) & 127) * 128u;
                const uint4 wc[1] = {w[i]};
                const uint32_t ec[1] = {e[i]}, a0[1] = {st0 + band}, a1[1] = {st1 + band};
                all &= dequant_slots<1, FAST>(wc, ec, a0, a1);
            }
        }
    }
    if constexpr (FAST) {
        if (static_cast<int32_t>(all) >= 0)              // a block with E >= 254: rare
            dequant_slab<C, false>(ln, raw_mant, raw_exp, dst_base, row_base, t, T_MA_rows);
    }
}

// A bundle of NS consecutive thin slabs (consecutive raw buffers, consecutive row ranges of one
// 128-row operand group): all loads first, then all conversions and stores, so that a thread has
// NS * DQ_ITERS slots in flight exactly as with one 128-row slab.
template <class C, int NS, bool FAST = true>
__device__ __forceinline__ void dequant_bundle(const DequantLane<C>& ln, uint32_t raw0, uint32_t raw_stride, uint32_t mant_bytes,
                                               uint32_t dst_base, int row_base0, int t, int slab_rows) {
    static_assert(C::SLOTS % C::GROUP_THREADS == 0, "whole iterations");
    const int r0 = t / C::SLOTS_PER_ROW;
    (void)r0;
    uint4 w[NS][C::DQ_ITERS];
    uint32_t e[NS][C::DQ_ITERS];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const uint32_t ld = raw0 + s * raw_stride + ln.ld_off, le = raw0 + s * raw_stride + mant_bytes + ln.exp_off;
#pragma unroll
        for (int i = 0; i < C::DQ_ITERS; ++i) {
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[s][i].x), "=r"(w[s][i].y), "=r"(w[s][i].z), "=r"(w[s][i].w)
                         : "r"(ld + static_cast<uint32_t>(i * C::GROUP_THREADS * 16)));
            uint16_t e2;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(e2) : "r"(le + static_cast<uint32_t>(i * C::ROWS_PER_ITER * 8)));
            e[s][i] = e2;
        }
    }
    constexpr int N = NS * C::DQ_ITERS;                  // at most 4: the whole bundle under one test
    uint4 wc[N];
    uint32_t ec[N], a0[N], a1[N];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const uint32_t st0 = dst_base + static_cast<uint32_t>(row_base0 + s * slab_rows) * 128u + ln.st_off0;
        const uint32_t st1 = dst_base + static_cast<uint32_t>(row_base0 + s * slab_rows) * 128u + ln.st_off1;
#pragma unroll
        for (int i = 0; i < C::DQ_ITERS; ++i) {
            constexpr uint32_t kBandRows = C::ROWS_PER_ITER;
            const uint32_t band = static_cast<uint32_t>((i * kBandRows) & 127) * 128u;     // thin slabs stay inside one group
            wc[s * C::DQ_ITERS + i] = w[s][i]; ec[s * C::DQ_ITERS + i] = e[s][i];
            a0[s * C::DQ_ITERS + i] = st0 + band; a1[s * C::DQ_ITERS + i] = st1 + band;
        }
    }
    const uint32_t all = dequant_slots<N, FAST>(wc, ec, a0, a1);
    if constexpr (FAST) {
        if (static_cast<int32_t>(all) >= 0)              // a block with E >= 254: rare
            dequant_bundle<C, NS, false>(ln, raw0, raw_stride, mant_bytes, dst_base, row_base0, t, slab_rows);
    }
}

// ---------------------------------------------------------------------------------------------
// The raw-A producer role of atb_gemm_kernel and atb_gemm_pair_kernel (one elected thread of a warp of its own:
// the raw slabs feed the dequantisers, which run ahead of the UMMAs, so these loads must not queue behind the
// wait for a free B stage).  Per work item of the CTA - next_item(it, row0, k_begin, k_end) gives the first row of
// this CTA's part of the item and its range of K-steps, false when the CTA has no more - it walks the 64-column
// rounds of the K range (upwards or downwards, see serpentine_k) and loads the C::SLABS slabs of
// C::SLAB_ROWS rows of each round: mantissa box and exponent box into one raw buffer, under one barrier.
// ---------------------------------------------------------------------------------------------
template <class C, class NextItem>
__device__ __forceinline__ void a_producer_role(const Ctx& cx, const CUtensorMap* tm_mant, const CUtensorMap* tm_exp,
                                                uint32_t raw_full, uint32_t raw_empty, uint32_t raw_base, NextItem&& next_item) {
    Cursor<C::NR, C::LR> rr;
    bool ok = true;
#ifndef ATB_NO_L2_HINTS
    // The tile walk keeps a band of A row panels in use wave after wave while the B column panels
    // change: A is asked to stay in the L2 longest.
    const uint64_t a_policy = l2_policy_evict_last();
#endif
    int row0 = 0, k_begin = 0, k_end = 0;
    for (int it = 0; ok && next_item(it, row0, k_begin, k_end); ++it) {
        for (int kh0 = k_begin * C::KH; ok && kh0 < k_end * C::KH; ++kh0) {      // 64-column rounds
            // (a downward walk keeps the rounds of a T_K = 128 step in their upward order)
            const int kh = serpentine_k(it, kh0 / C::KH, k_begin, k_end) * C::KH + kh0 % C::KH;
            for (int s = 0; s < C::SLABS; ++s) {
                // (a barrier of this CTA alone, on a CTA pair too)
                if (!(ok = wait_bar_spin(cx, raw_empty + 8 * rr.freed_bar(), rr.freed_parity(), 0x002))) break;
                const uint32_t fr = raw_full + 8 * rr.bar;
                const uint32_t dst = raw_base + rr.buf() * C::RAW_BYTES;
#ifdef ATB_PROFILE
                const long long issue_t0 = clock64();
#endif
                mbar_arrive_expect_tx(fr, C::RAW_BYTES);
#ifndef ATB_NO_L2_HINTS
                tma_load_2d_hint(dst, tm_mant, kh * kKA, row0 + s * C::SLAB_ROWS, fr, a_policy);
                tma_load_2d_hint(dst + C::RAW_MANT_BYTES, tm_exp, row0 + s * C::SLAB_ROWS, kh, fr, a_policy);
#else
                tma_load_2d(dst, tm_mant, kh * kKA, row0 + s * C::SLAB_ROWS, fr);
                tma_load_2d(dst + C::RAW_MANT_BYTES, tm_exp, row0 + s * C::SLAB_ROWS, kh, fr);
#endif
#ifdef ATB_PROFILE      // slot 3: cycles this thread spent issuing the loads of A
                atomicAdd(&g_wait_cycles[blockIdx.x & 255][3], static_cast<unsigned long long>(clock64() - issue_t0));
#endif
                rr.template advance<1>();
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The dequantiser role of atb_gemm_kernel and atb_gemm_pair_kernel: one warp of dequantiser group
// `my_group` (thread `t` of the group).  The group does not need to know tiles or K-steps: slabs arrive in
// ring order, so it takes every DQ_GROUPS-th bundle of the CTA's stream of `my_slabs` raw slabs, waits for the
// raw slabs and for a free place in the operand ring, converts, and hands the operand on.
// C: the kernel's compile-time configuration (slab height SLAB_ROWS, bundle, ring depths and barrier counts).
// PAIR: the operand is announced on the leader CTA's barrier and the waits use cluster-scope acquire.
// ---------------------------------------------------------------------------------------------
template <class C, bool PAIR>
__device__ __forceinline__ void dequantiser_role(const Ctx& cx, int t, int my_group, int warp, int lane, int64_t my_slabs,
                                                 uint32_t raw_full, uint32_t raw_empty, uint32_t deq_full, uint32_t deq_empty,
                                                 uint32_t raw_base, uint32_t deq_base) {
    constexpr int SLAB = C::SLAB_ROWS;
    const DequantLane<C> ln(t, SLAB);
#ifdef ATB_PROFILE_SKIP_DEQUANT
    // diagnostic: the operand ring holds fixed pseudo-random bf16 values (zeros would lower the
    // tensor cores' power and flatter the clock)
    for (uint32_t i = threadIdx.x - kFirstDequantWarp * 32; i < C::NG * C::GROUP_BYTES / 4; i += kDequantWarps * 32) {
        uint32_t h = (i + 1u) * 2654435761u; h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        const uint32_t v = (h & 0x807F807Fu) | 0x3F003F00u;          // +-[0.5, 1) in both halves
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(deq_base + i * 4), "r"(v) : "memory");
    }
    fence_proxy_async_smem();
#endif
    Cursor<C::NR, C::LR> rr;
    Cursor<C::ND, C::LD> rd;
    rr.start_at(my_group * C::BUNDLE);
    rd.start_at(my_group);
    for (int64_t n = static_cast<int64_t>(my_group) * C::BUNDLE; n < my_slabs; n += C::DQ_GROUPS * C::BUNDLE) {
        bool ok = true;
#pragma unroll
        for (int i = 0; i < C::BUNDLE; ++i)        // bars and buffers of a bundle are consecutive
            ok = ok && wait_bar_t<false, false>(cx, raw_full + 8 * (rr.bar + i), rr.phase, 0x301);     // filled by this CTA's own TMA loads
        ok = ok && wait_bar_t<false, PAIR>(cx, deq_empty + 8 * rd.freed_bar(), rd.freed_parity(), 0x302);
        if (!ok) break;
#ifndef ATB_PROFILE_SKIP_DEQUANT    // diagnostic: the pipeline without the conversion work (results are wrong)
        // all slots of the bundle in flight at once where that is at most four per thread (registers)
        if constexpr (C::BUNDLE > 1 && C::SLOTS % C::GROUP_THREADS == 0 && C::BUNDLE * C::DQ_ITERS <= 4) {
            dequant_bundle<C, C::BUNDLE>(ln, raw_base + rr.buf() * C::RAW_BYTES, C::RAW_BYTES, C::RAW_MANT_BYTES,
                                         deq_base + (rd.buf() / C::SPB) * C::GROUP_BYTES, (rd.buf() % C::SPB) * C::BUNDLE * SLAB, t, SLAB);
        } else {
#pragma unroll
            for (int i = 0; i < C::BUNDLE; ++i) {
                const uint32_t raw = raw_base + (rr.buf() + i) * C::RAW_BYTES;
                const uint32_t dst_base = deq_base + (SLAB <= 128 ? rd.buf() / C::SPB : rd.buf() * C::GPS) * C::GROUP_BYTES;
                dequant_slab<C>(ln, raw, raw + C::RAW_MANT_BYTES, dst_base,
                                SLAB <= 128 ? ((rd.buf() % C::SPB) * C::BUNDLE + i) * SLAB : 0, t, SLAB);
            }
        }
#endif
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            if constexpr (PAIR) {
                // CTA-scope release: the operand this publishes stays in this CTA's shared memory and is
                // read by this CTA's tensor core (after the proxy fence above) once the leader has seen
                // the arrival and issued the UMMA.  A cluster-scope release here kept a quarter of the
                // dequantiser warps in membar stalls (ncu) and cost 1-2 %.  The waiter acquires at cluster
                // scope, so by the letter of the PTX memory model this release/acquire pair does not
                // synchronise; it is kept because no thread of the other CTA reads what is published (a
                // bit-for-bit soak of all slab heights against the single-CTA kernel stands in the test
                // suite).  -DATB_PAIR_RELEASE_CLUSTER builds the conforming form.
#ifdef ATB_PAIR_RELEASE_CLUSTER
                mbar_arrive_cluster(mapa_shared(deq_full + 8 * rd.bar, 0));
#else
                mbar_arrive_cluster_cta_release(mapa_shared(deq_full + 8 * rd.bar, 0));
#endif
            } else {
#ifdef ATB_TEST_WITHHOLD_DEQ_ARRIVAL
                // Test build of the timeout path only: the first dequantiser warp of CTA 0 keeps back its very
                // first arrival, so the issuer's bounded wait for that operand runs out, the CTA aborts, every
                // role returns and atb_device_status reports it.  No UMMA or copy depends on the missing arrival.
                if (!(blockIdx.x == 0 && warp == kFirstDequantWarp && n == 0))
#endif
                mbar_arrive(deq_full + 8 * rd.bar);
            }
#pragma unroll
            for (int i = 0; i < C::BUNDLE; ++i) mbar_arrive(raw_empty + 8 * (rr.bar + i));
        }
        rr.template advance<C::DQ_GROUPS * C::BUNDLE>();
        rd.template advance<C::DQ_GROUPS>();
    }
    (void)warp;
}

// ---------------------------------------------------------------------------------------------
// Epilogues of one warp: N_COLS accumulator columns of its 32 TMEM lanes (rows row0 .. row0+31,
// columns col0 ..) -> C.  `box` is the warp's staging in shared memory.
// ---------------------------------------------------------------------------------------------
// BF16 C: tcgen05.ld -> round to bf16 (RNE) -> swizzled box of 32 rows x BOX_COLS columns in shared
// memory -> global memory.  BOX_COLS = 64: 128-byte rows (4 KB); 32: 64-byte rows (2 KB).
// The accumulator is read 32 columns at a time; the load of the next 32 columns is issued as soon as
// the current ones are packed to bf16, so that its latency passes behind the staging and the stores.
// Two ways out of the box (measured: the single-CTA kernels are faster with the TMA store - one instruction in a
// warp that competes with the dequantisers for issue slots -, and so is the stacked form of the CTA-pair kernel,
// whose drain runs beside the next tile's K loop; the CTA-pair kernel's 256 x 512 tile, whose 128 x 512 accumulator
// per SM takes longest to drain and holds up the next tile meanwhile, is faster with direct stores: +4 % at
// K = 1024, +1 % at K = 8192):
//   TMA store   one instruction per box; costs about 5.5 cycles per row whatever the row carries (23 B per
//               cycle and SM at 128-byte rows, half of that at 64-byte rows); edges are clipped by the tensor map.
//   direct      the warp reads the box back row-wise and writes 16-byte chunks: 8 (4) lanes cover one row
//               segment, so every store instruction writes full 128-byte (64-byte) runs; rows and columns
//               beyond M, N are skipped (N is a multiple of 8: a 16-byte chunk is inside or outside).
#ifndef ATB_EPILOGUE_DIRECT          // tuning builds: -DATB_EPILOGUE_DIRECT=0|1, -DATB_EPILOGUE_DIRECT_PAIR=0|1
#define ATB_EPILOGUE_DIRECT 0
#endif
#ifndef ATB_EPILOGUE_DIRECT_PAIR
#define ATB_EPILOGUE_DIRECT_PAIR 1
#endif
template <int N_COLS, int BOX_COLS = 64, bool DIRECT = (ATB_EPILOGUE_DIRECT != 0)>
__device__ __forceinline__ void epilogue_bf16(const CUtensorMap* tm_c, __nv_bfloat16* __restrict__ C, int64_t ldc, uint32_t t_addr,
                                              uint32_t box, int lane, int row0, int col0, int64_t M, int64_t N) {
    static_assert(BOX_COLS == 64 || BOX_COLS == 32, "box width");
    constexpr int CPR = BOX_COLS / 8;                  // 16-byte chunks per row of the box
    constexpr int RPI = 32 / CPR;                      // rows one store instruction of the warp covers (direct)
    constexpr uint32_t kSwMask = CPR - 1;
    constexpr int HALVES = BOX_COLS / 32, N_LOADS = N_COLS / 32;
    const uint32_t my_row = box + lane * (BOX_COLS * 2);
    const uint32_t sw = BOX_COLS == 64 ? static_cast<uint32_t>(lane & 7) : (static_cast<uint32_t>(lane >> 1) & 3u);
    const int och = lane % CPR, orow = lane / CPR;     // direct: this lane copies chunk och of rows orow, orow + RPI, ...
#ifndef ATB_NO_L2_HINTS
    const uint64_t store_policy = l2_policy_evict_first();   // C is not read again: first to leave the L2
#endif
    uint32_t v[32];
    tmem_ld_32x32b_x32(t_addr, v);
#pragma unroll 1
    for (int l = 0; l < N_LOADS; ++l) {
        const int c = l / HALVES, h = l % HALVES;
        tmem_ld_wait_for(v);
        uint32_t o[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
            o[e] = *reinterpret_cast<uint32_t*>(&b2);
        }
        if (l + 1 < N_LOADS) tmem_ld_32x32b_x32(t_addr + (l + 1) * 32, v);       // in flight during what follows
        if (h == 0) {
            // the box is free again: the TMA store that read it has finished / every lane has copied its part out
            if constexpr (!DIRECT) { if (lane == 0) tma_store_wait_read<0>(); }
            __syncwarp();
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + ((static_cast<uint32_t>(h * 4 + j) ^ sw) << 4)),
                         "r"(o[4 * j]), "r"(o[4 * j + 1]), "r"(o[4 * j + 2]), "r"(o[4 * j + 3]) : "memory");
        if (h != HALVES - 1) continue;
        if constexpr (!DIRECT) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && row0 < M && col0 + c * BOX_COLS < N) {   // rows / columns past the edge are clipped
#ifndef ATB_NO_L2_HINTS
                tma_store_2d_hint(tm_c, box, col0 + c * BOX_COLS, row0, store_policy);
#else
                tma_store_2d(tm_c, box, col0 + c * BOX_COLS, row0);
#endif
                tma_store_commit();
            }
        } else {
            __syncwarp();
            const int64_t col = static_cast<int64_t>(col0) + c * BOX_COLS + och * 8;
            __nv_bfloat16* dst = C + (static_cast<int64_t>(row0) + orow) * ldc + col;
            const int rows_left = static_cast<int>(min(M - row0 - orow, static_cast<int64_t>(32)));     // rows r < rows_left exist
            uint32_t src = box + static_cast<uint32_t>(orow) * (BOX_COLS * 2);
#pragma unroll
            for (int i = 0; i < CPR; ++i) {
                // row r = i * RPI + orow: with 64-byte rows RPI = 8 and r's swizzle term is orow's; with 128-byte rows RPI = 4
                const uint32_t rsw = BOX_COLS == 64 ? static_cast<uint32_t>((i * RPI + orow) & 7) : (static_cast<uint32_t>(orow >> 1) & 3u);
                uint32_t o0, o1, o2, o3;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(o0), "=r"(o1), "=r"(o2), "=r"(o3)
                             : "r"(src + (((static_cast<uint32_t>(och) ^ rsw) & kSwMask) << 4)));
                if (i * RPI < rows_left && col < N) {
#ifndef ATB_NO_L2_HINTS
                    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst), "r"(o0), "r"(o1), "r"(o2), "r"(o3),
                                 "l"(store_policy) : "memory");
#else
                    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
#endif
                }
                dst += static_cast<int64_t>(RPI) * ldc;
                src += RPI * (BOX_COLS * 2);
            }
        }
    }
}

// BFP16 C: a thread owns one row; per 64 columns it quantises 8 blocks of 8 FP32 accumulators
// (exactly as atb_quantize_bfp16 would), stages the 64 mantissa bytes of its row in a 32 x 64-byte
// box (64-byte swizzle) for one TMA store, and writes the 8 exponents - contiguous in the exponent
// plane [ceil(N/64)][exp_rows][8], rows adjacent - directly.  Rows of the plane's padding
// (M <= row < exp_rows) get exponent 0.
template <int N_COLS>
__device__ __forceinline__ void epilogue_bfp16(const CUtensorMap* tm_c, uint32_t t_addr, uint32_t box, int lane, int row0,
                                               int col0, int64_t M, int64_t N, uint8_t* exp_plane, int64_t exp_rows) {
    const uint32_t my_row64 = box + lane * 64;
    const uint32_t sw64 = static_cast<uint32_t>(lane >> 1) & 3u;
    const int64_t row = static_cast<int64_t>(row0) + lane;
#pragma unroll 1
    for (int c = 0; c < N_COLS / 64; ++c) {
        if (lane == 0) tma_store_wait_read<0>();
        __syncwarp();
        uint32_t e_lo = 0, e_hi = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_addr + c * 64 + h * 32, v);
            tmem_ld_wait();
            uint32_t m8[8];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] = __uint_as_float(v[b * 8 + e]);
                uint32_t pk[2];
                const uint32_t E = static_cast<uint32_t>(bfp16::quantize_block8(x, pk));
                m8[2 * b] = pk[0];
                m8[2 * b + 1] = pk[1];
                if (h == 0) e_lo |= E << (8 * b); else e_hi |= E << (8 * b);
            }
#pragma unroll
            for (int j = 0; j < 2; ++j)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(my_row64 + ((static_cast<uint32_t>(h * 2 + j) ^ sw64) << 4)),
                             "r"(m8[4 * j]), "r"(m8[4 * j + 1]), "r"(m8[4 * j + 2]), "r"(m8[4 * j + 3]) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
        const int64_t col = static_cast<int64_t>(col0) + c * 64;
        if (col < N) {
            if (lane == 0 && row0 < M) {
                tma_store_2d(tm_c, box, static_cast<int>(col), row0);
                tma_store_commit();
            }
            if (row < exp_rows) {
                const bool real = row < M;
                uint2 ev = make_uint2(real ? e_lo : 0u, real ? e_hi : 0u);
                *reinterpret_cast<uint2*>(exp_plane + ((col >> 6) * exp_rows + row) * 8) = ev;
            }
        }
    }
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

bool make_map_2d(CUtensorMap* map, CUtensorMapDataType type, uint32_t elem_bytes, const void* base,
                 uint64_t dim0, uint64_t dim1, uint64_t stride1_bytes, uint32_t box0, uint32_t box1,
                 CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {dim0, dim1};
    const cuuint64_t strides[1] = {stride1_bytes};
    const cuuint32_t box[2] = {box0, box1};
    const cuuint32_t estr[2] = {1, 1};
    (void)elem_bytes;
    return fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
