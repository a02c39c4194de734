// Internal helpers shared by the library's translation units (not part of the ABI).
#pragma once
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "atb.h"

namespace atb {

// Records the detail string of the calling thread's failing call and returns `status`.
atb_status_t fail(atb_status_t status, const char* fmt, ...);
void clear_error();

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shared-memory plan of the GEMM kernel for one tiling (host side; the kernel receives it).
struct GemmPlan {
    int n_b_stages;      // B-tile ring depth
    int n_groups;        // dequantised-A ring depth, in 128-row groups
    int n_raw_stages;    // raw (BFP16) A-slab ring depth
    int dq_groups;       // dequantiser warp groups
    int acc_bufs;        // accumulator buffers in TMEM (1 or 2)
    int tmem_cols;       // allocated TMEM columns (power of two)
    uint32_t smem_bytes; // dynamic shared memory of the launch
};
// Fills `plan`; false if the tiling is not supported or does not fit.  `single_cta` asks for the one-CTA
// plan of a tiling that normally runs as stacked tiles on a CTA pair (see is_stacked_pair_tiling).
bool plan_gemm(int T_MA, int T_MC, int T_K, int T_N, GemmPlan* plan, bool single_cta = false);
// True for the tiling whose 256 x 512 tile is computed by a CTA pair (cluster of 2): T_MC = 256, T_N = 512, T_K = 64.
inline bool is_pair_tiling(int T_MC, int T_K, int T_N) { return T_MC == 256 && T_N == 512 && T_K == 64; }
// True for the tiling whose 128 x 256 tiles are computed two at a time, one above the other, by a CTA pair
// that shares every B tile between them: T_MC = 128, T_N = 256, T_K = 128 (atb_gemm, where M > 128; a problem of
// one tile row and the split-K and BFP16-output entry points run it on single CTAs).
inline bool is_stacked_pair_tiling(int T_MC, int T_K, int T_N) { return T_MC == 128 && T_N == 256 && T_K == 128; }
// T_N = 512: the 256 x 512 pair tile; T_N = 256: two stacked 128 x 256 tiles.
atb_status_t launch_gemm_pair(int T_MA, int T_N, const GemmPlan& plan, int64_t M, int64_t N, int64_t K, const int8_t* mant,
                              const uint8_t* exp, const void* B, int64_t ldb, void* C, int64_t ldc, int num_sms,
                              unsigned int* error_flag, void* stream, uint8_t* C_exp = nullptr);

// Thin slabs (T_MA < 128) are converted in bundles: the largest power-of-two number of consecutive
// slabs, at most spg = 128 / T_MA (one operand group), such that the raw ring of n_raw slabs holds a
// whole bundle for every one of the `groups` dequantiser groups.
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int slab_bundle(int spg, int n_raw, int groups) {
    int b = spg;
    while (b > 1 && n_raw % (b * groups)) b >>= 1;
    return b;
}

// Reads and clears the timeout flag of the precision-configuration kernels (0 = none).
unsigned int take_cfg_error_flag();

}  // namespace atb
