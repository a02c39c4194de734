// CPU oracle for the BFP16 x BF16 GEMM hot path.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain reference that the CUDA library is checked
// against.  Only the test-suite, the smoke check and the benchmark's
// cpu_baseline / reference arm may build, load or call it; the product library
// never does, and the two share no code, headers, tables or helpers.
//
// What it computes (everything in FP64 unless stated):
//   * BFP16 quantisation of an fp32 matrix: blocks of 8 consecutive K-elements
//     share one 8-bit exponent and carry 8-bit mantissas (Section 2.4 gives the
//     format: 8 values, one 8-bit exponent, 8-bit mantissas, 9 bytes).  The
//     paper does not say how the exponent is chosen or how mantissas are
//     rounded; the readings taken here are listed at each function.
//   * Dequantisation  a = m * 2^(E-133).
//   * The GEMM as its plain definition, C[i][j] = sum_k a[i][k]*b[k][j]
//     (Section 1: C = A x B), because asymmetric tile buffering (Section 3)
//     only changes buffer lifetimes, not the result.  S[i][j] = sum_k |a*b| is
//     produced beside it for the error bound.
//   * The per-element acceptance test
//        |C_gpu - C_ref| <= 2^-7 |C_ref| + 2^-12 S.
//
// Logical layouts (row-major, no padding unless a leading dimension is given):
//   mant[M][K] int8, exp[M][K/8] uint8, B[K][N] bf16 as uint16 bit patterns.
//
// Parity status: quantiser, dequantiser, GEMM and acceptance test are pinned by
// the not-gpu tests (exact-rational brute force, hand-worked blocks, integer
// and permutation matrices, library matmul).  Agreement of the quantiser with
// AMD's own BFP16 tooling is unpinned: the paper gives no algorithm or example.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double bf16_bits_to_double(uint16_t h) {
    uint32_t w = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &w, sizeof f);
    return static_cast<double>(f);
}

// Shared exponent of one block: the biased fp32 exponent of the largest
// magnitude (NaNs ignored), 0 when that magnitude is zero or subnormal,
// capped at 254 (so +-Inf maps to 254).
inline int block_exponent(const float* x) {
    double amax = 0.0;
    for (int t = 0; t < 8; ++t) {
        double v = std::fabs(static_cast<double>(x[t]));
        if (v != v) continue;              // NaN: ignored
        if (v > amax) amax = v;
    }
    if (amax == 0.0) return 0;
    if (std::isinf(amax)) return 254;
    int e2;
    std::frexp(amax, &e2);                 // amax = f * 2^e2, f in [0.5,1)
    int E = (e2 - 1) + 127;                // floor(log2 amax) + bias
    if (E < 1) E = 0;                      // below the smallest normal fp32
    if (E > 254) E = 254;
    return E;
}

// Mantissa of one element at block exponent E: round-to-nearest-even of
// x / 2^(E-133), saturated to [-127, 127]; NaN -> 0; +-Inf -> +-127.
inline int element_mantissa(float x, int E) {
    double v = static_cast<double>(x);
    if (v != v) return 0;
    if (std::isinf(v)) return v > 0 ? 127 : -127;
    double q = std::ldexp(v, 133 - E);     // exact power-of-two scaling in FP64
    double r = std::nearbyint(q);          // default rounding mode: ties to even
    if (r > 127.0) r = 127.0;
    if (r < -127.0) r = -127.0;
    return static_cast<int>(r);
}

}  // namespace

extern "C" {

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Quantise A[M][K] (fp32, leading dimension lda) to BFP16 planes.
// Returns 0, or -1 when K is not a multiple of 8.
int oracle_quantize_bfp16(const float* A, int64_t M, int64_t K, int64_t lda,
                          int8_t* mant, uint8_t* exp) {
    if (K % 8 != 0 || M < 0 || K < 0) return -1;
    const int64_t KB = K / 8;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t kb = 0; kb < KB; ++kb) {
            const float* x = A + i * lda + kb * 8;
            const int E = block_exponent(x);
            exp[i * KB + kb] = static_cast<uint8_t>(E);
            for (int t = 0; t < 8; ++t)
                mant[i * K + kb * 8 + t] = static_cast<int8_t>(element_mantissa(x[t], E));
        }
    }
    return 0;
}

// a[i][k] = m * 2^(E-133), exact in FP64.
void oracle_dequantize_f64(const int8_t* mant, const uint8_t* exp, int64_t M, int64_t K,
                           double* out) {
    const int64_t KB = K / 8;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t k = 0; k < K; ++k)
            out[i * K + k] = std::ldexp(static_cast<double>(mant[i * K + k]),
                                        static_cast<int>(exp[i * KB + k / 8]) - 133);
}

// Rows rows[0..n_rows) of C = dequant(A) x B and of S = sum_k |a*b|, FP64,
// k ascending.  Output row r of C_out / S_out (each [n_rows][N]) holds
// logical row rows[r].  rows == nullptr means rows 0..n_rows-1.
void oracle_gemm_rows_f64(int64_t N, int64_t K, const int8_t* mant, const uint8_t* exp,
                          const uint16_t* B, int64_t ldb, const int64_t* rows, int64_t n_rows,
                          double* C_out, double* S_out) {
    const int64_t KB = K / 8;
    std::vector<double> Bd(static_cast<size_t>(K) * N);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < K; ++k)
        for (int64_t j = 0; j < N; ++j) Bd[k * N + j] = bf16_bits_to_double(B[k * ldb + j]);

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t i = rows ? rows[r] : r;
        double* c = C_out + r * N;
        double* s = S_out ? S_out + r * N : nullptr;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s)
            for (int64_t j = 0; j < N; ++j) s[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = std::ldexp(static_cast<double>(mant[i * K + k]),
                                        static_cast<int>(exp[i * KB + k / 8]) - 133);
            const double aa = std::fabs(a);
            const double* b = &Bd[k * N];
            for (int64_t j = 0; j < N; ++j) c[j] += a * b[j];
            if (s)
                for (int64_t j = 0; j < N; ++j) s[j] += aa * std::fabs(b[j]);
        }
    }
}

// Full GEMM: all M rows.
void oracle_gemm_f64(int64_t M, int64_t N, int64_t K, const int8_t* mant, const uint8_t* exp,
                     const uint16_t* B, int64_t ldb, double* C, double* S) {
    oracle_gemm_rows_f64(N, K, mant, exp, B, ldb, nullptr, M, C, S);
}

// Acceptance test over an [n_rows][N] block: C_gpu (bf16 bits, leading
// dimension ldc) against C_ref/S (FP64, dense).  An element passes iff it is
// finite and |C_gpu - C_ref| <= 2^-7 |C_ref| + 2^-12 S.  Returns the number of
// failing elements; *max_ratio receives max(error / bound) (bound 0 with error
// 0 counts as ratio 0; bound 0 with error > 0 as +inf).
int64_t oracle_check_tolerance(const uint16_t* C_gpu, int64_t ldc, const double* C_ref,
                               const double* S, int64_t n_rows, int64_t N, double* max_ratio) {
    int64_t bad = 0;
    double worst = 0.0;
    for (int64_t r = 0; r < n_rows; ++r) {
        for (int64_t j = 0; j < N; ++j) {
            const double g = bf16_bits_to_double(C_gpu[r * ldc + j]);
            const double ref = C_ref[r * N + j];
            const double bound = std::ldexp(std::fabs(ref), -7) + std::ldexp(S[r * N + j], -12);
            double ratio;
            if (!std::isfinite(g)) {
                ratio = INFINITY;
            } else {
                const double err = std::fabs(g - ref);
                ratio = (err == 0.0) ? 0.0 : (bound > 0.0 ? err / bound : INFINITY);
            }
            if (!(ratio <= 1.0)) ++bad;
            if (ratio > worst || ratio != ratio) worst = ratio;
        }
    }
    if (max_ratio) *max_ratio = worst;
    return bad;
}

}  // extern "C"
