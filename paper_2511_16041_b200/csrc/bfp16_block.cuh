// Quantisation of one BFP16 block (8 fp32 values sharing an 8-bit exponent, int8 mantissas; format of
// Section 2.4) in registers.  Used by the quantiser kernel and by the quantising GEMM epilogue.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace bfp16 {

__device__ __forceinline__ float pow2f(int e) {   // 2^e for e in [-126, 127]
    return __uint_as_float(static_cast<uint32_t>(e + 127) << 23);
}

// E = biased fp32 exponent of the largest magnitude (NaNs do not take part; 0 for a zero or subnormal
// maximum; 254 at most, which also covers infinities); m = RNE(x / 2^(E-133)) saturated to +-127,
// NaN -> 0.  Returns E; packed[0] holds m_0..m_3 and packed[1] m_4..m_7, one byte each, low first.
__device__ __forceinline__ int quantize_block8(const float (&x)[8], uint32_t (&packed)[2]) {
    uint32_t amax_bits = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        uint32_t b = __float_as_uint(x[t]) & 0x7FFFFFFFu;
        if (b > 0x7F800000u) b = 0;
        amax_bits = max(amax_bits, b);
    }
    int E = static_cast<int>(amax_bits >> 23);
    E = min(E, 254);
    // x / 2^(E-133) as two exact power-of-two multiplications (one factor alone would leave the
    // fp32 range at both ends of E).
    const int sh = 133 - E;
    const int sa = sh >> 1, sb = sh - sa;
    const float fa = pow2f(sa), fb = pow2f(sb);
    packed[0] = 0u;
    packed[1] = 0u;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const float q = (x[t] * fa) * fb;
        int r = __float2int_rn(q);            // ties to even; NaN -> 0; +-Inf saturate
        r = max(-127, min(127, r));
        packed[t >> 2] |= (static_cast<uint32_t>(r) & 0xFFu) << (8 * (t & 3));
    }
    return E;
}

}  // namespace bfp16
