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
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kDequantWarps = 16;
constexpr int kThreads = (7 + kDequantWarps) * 32;      // + B producer, UMMA issuer, 4 epilogue warps, A producer
constexpr int kAProducerWarp = 6 + kDequantWarps;       // the last warp
// The dequantiser warps work in groups; slabs are dealt to the groups in turn, so that several
// slabs are in flight and every thread has a few 16-element slots per barrier round trip.
// Ring depths are multiples of the group count: a ring stage is then always served by the same
// group, which keeps each mbarrier's phases strictly in order for its waiters.
__host__ __device__ constexpr int dq_groups(int T_MA, int T_K, int T_N) {
#ifdef ATB_DQ_GROUPS
    return ATB_DQ_GROUPS;
#else
    // two groups for big slabs, and where a double-buffered B tile already takes 128 KB
    return (T_MA * T_K >= 256 * 64 || T_K * T_N >= 128 * 256) ? 2 : 4;
#endif
}
constexpr int kFirstEpilogueWarp = 2;
constexpr int kFirstDequantWarp = 6;
constexpr int kMaxStages = 16;
constexpr uint32_t kEpilogueBoxBytes = 32 * 128;   // 32 rows x 64 bf16 columns
constexpr uint32_t kSmemBudget = 232448;          // 227 KB of dynamic shared memory per CTA
constexpr uint64_t kWaitTimeoutNs = 2000000000ull;  // every mbarrier wait gives up after 2 s

struct GemmParams {
    int64_t M, N, K, ldc;
    __nv_bfloat16* C;
    int m_tiles, n_tiles, k_steps;
    int n_b_stages, n_groups, n_raw_stages, acc_bufs, tmem_cols;
    unsigned int* error_flag;
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
    // `step` stages at once; n is a multiple of step and stage stays congruent modulo step
    __device__ __forceinline__ void advance_by(int step, int n) {
        stage += step;
        if (stage >= n) { stage -= n; phase ^= 1u; }
    }
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

__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int& mt, int& nt) {
    // Bands of 16 tile-rows, column-major inside a band: the CTAs of one wave share a few
    // A row-panels and B column-panels in L2.
    const int per_band = 16 * n_tiles;
    const int band = tile / per_band, i = tile - band * per_band;
    const int rows = min(16, m_tiles - band * 16);
    mt = band * 16 + i % rows;
    nt = i / rows;
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
//      (h >> 3) + 0x3800 per half, done for both halves by one mad.hi.u32 (x * 2^29 >> 32).
//   3. add.bf16x2 subtracts 128 (m, exact: 7 significant bits), mul.bf16x2 scales by the block's
//      2^(E-133) (from a 256-entry table of packed bf16 pairs: normal for E >= 7, bf16-subnormal
//      below); the product is exact for every E, subnormal results included.
// Only the prmt runs on the integer ALU pipe - the pipe the dequantisers saturate first; the other
// four operations go to the FMA pipe.
__device__ __forceinline__ uint32_t dequant_pair(uint32_t u, uint32_t selector, uint32_t scale2) {
    const uint32_t h2 = __byte_perm(u, 0x64646464u, selector);
    uint32_t t, b, d, r;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(t) : "r"(h2), "r"(0xE400E400u));          // - 1024
    asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(b) : "r"(t), "r"(0x20000000u), "r"(0x38003800u));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(b), "r"(0xC300C300u));          // - 128
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(d), "r"(scale2));
    return r;
}

// Table entry for exponent E: 2^(E-133) as bf16, in both halves of the word.
__device__ __forceinline__ uint32_t scale_table_entry(uint32_t E) {
    const uint32_t bits = (E >= 7u) ? ((E - 6u) << 7) : (1u << E);
    return E == 255u ? 0u : bits * 0x10001u;
}

template <class C>
__device__ __forceinline__ void dequant_slab(uint32_t raw_mant, uint32_t raw_exp, uint32_t scale_lut,
                                             uint32_t dst_base, int row_base, int t, int T_MA_rows) {
    const int p = t % C::SLOTS_PER_ROW;                 // blocks 2p, 2p + 1 of the row
    const int r0 = t / C::SLOTS_PER_ROW;
    const int kb = 2 * p;
    uint4 w[C::DQ_ITERS];
    uint32_t e[C::DQ_ITERS];
#pragma unroll
    for (int i = 0; i < C::DQ_ITERS; ++i) {
        const int r = r0 + i * C::ROWS_PER_ITER;
        if (C::SLOTS % C::GROUP_THREADS == 0 || r < T_MA_rows) {
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[i].x), "=r"(w[i].y), "=r"(w[i].z), "=r"(w[i].w)
                         : "r"(raw_mant + (r * C::SLOTS_PER_ROW + p) * 16));
            uint16_t e2;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(e2)
                         : "r"(raw_exp + (kb >> 3) * T_MA_rows * 8 + r * 8 + (kb & 7)));
            e[i] = e2;
        }
    }
#pragma unroll
    for (int i = 0; i < C::DQ_ITERS; ++i) {
        const int r = r0 + i * C::ROWS_PER_ITER;
        if (C::SLOTS % C::GROUP_THREADS == 0 || r < T_MA_rows) {
            uint32_t s0, s1;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(s0) : "r"(scale_lut + (e[i] & 0xFFu) * 4));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(s1) : "r"(scale_lut + (e[i] >> 8) * 4));
            const uint32_t u0 = w[i].x ^ 0x80808080u, u1 = w[i].y ^ 0x80808080u;
            const uint32_t u2 = w[i].z ^ 0x80808080u, u3 = w[i].w ^ 0x80808080u;
            const int rr = row_base + r;
            const uint32_t row_addr = dst_base + (rr >> 7) * C::GROUP_BYTES + (kb >> 3) * C::KHALF_BYTES + (rr & 127) * 128;
            const uint32_t sw = static_cast<uint32_t>(rr & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + ((((kb & 7)) ^ sw) << 4)),
                         "r"(dequant_pair(u0, 0x4140u, s0)), "r"(dequant_pair(u0, 0x4342u, s0)),
                         "r"(dequant_pair(u1, 0x4140u, s0)), "r"(dequant_pair(u1, 0x4342u, s0))
                         : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + ((((kb & 7) + 1) ^ sw) << 4)),
                         "r"(dequant_pair(u2, 0x4140u, s1)), "r"(dequant_pair(u2, 0x4342u, s1)),
                         "r"(dequant_pair(u3, 0x4140u, s1)), "r"(dequant_pair(u3, 0x4342u, s1))
                         : "memory");
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
