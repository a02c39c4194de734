// Quantisation of one BFP16 block (8 fp32 values sharing an 8-bit exponent, int8 mantissas; format of
// Section 2.4) in registers.  Used by the quantiser kernel and by the quantising GEMM epilogue.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace bfp16 {

__device__ __forceinline__ float pow2f(int e) {   // 2^e for e in [-126, 127]
    return __uint_as_float(static_cast<uint32_t>(e + 127) << 23);
}

// Packs RNE(q_0) .. RNE(q_3), saturated to [-127, 127], into the four bytes of a word, q_0 lowest.
// cvt.rni.s32.f32 gives 0 for NaN and the extreme integers for +-Inf; cvt.pack.sat saturates two integers to
// [-128, 127], puts them into the low half (first operand above second) and moves the low half of its
// third operand to the top; a byte of -128 (from q in [-128.5, -127.5]) is then moved to -127.
__device__ __forceinline__ uint32_t pack_mantissas4(float q0, float q1, float q2, float q3) {
    const int r0 = __float2int_rn(q0), r1 = __float2int_rn(q1), r2 = __float2int_rn(q2), r3 = __float2int_rn(q3);
    uint32_t hi, p;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(r3), "r"(r2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(p) : "r"(r1), "r"(r0), "r"(hi));
    // a byte equals 0x80 iff its top bit is set and its low seven bits are zero
    const uint32_t low7_nonzero = ((p & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) & 0x80808080u;
    const uint32_t is_m128 = p & 0x80808080u & ~low7_nonzero;
    return p | (is_m128 >> 7);
}

// E = biased fp32 exponent of the largest magnitude (NaNs do not take part; 0 for a zero or subnormal
// maximum; 254 at most, which also covers infinities); m = RNE(x / 2^(E-133)) saturated to +-127,
// NaN -> 0.  Returns E; packed[0] holds m_0..m_3 and packed[1] m_4..m_7, one byte each, low first.
__device__ __forceinline__ int quantize_block8(const float (&x)[8], uint32_t (&packed)[2]) {
    // largest magnitude: fmaxf passes over NaNs (it returns the other operand); a block of NaNs only is a zero block
    float amax = fmaxf(fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3]))),
                       fmaxf(fmaxf(fabsf(x[4]), fabsf(x[5])), fmaxf(fabsf(x[6]), fabsf(x[7]))));
    uint32_t amax_bits = __float_as_uint(amax);
    if (amax_bits > 0x7F800000u) amax_bits = 0;
    const int E = min(static_cast<int>(amax_bits >> 23), 254);
    const int sh = 133 - E;                        // x / 2^(E-133) = x * 2^sh, an exact scaling
    if (sh <= 127) {
        // one factor (E >= 6, i.e. all but blocks below 2^-121): a product that leaves the normal range is
        // below one half in magnitude and rounds to 0 either way
        const float f = pow2f(sh);
        packed[0] = pack_mantissas4(x[0] * f, x[1] * f, x[2] * f, x[3] * f);
        packed[1] = pack_mantissas4(x[4] * f, x[5] * f, x[6] * f, x[7] * f);
    } else {
        // two exact power-of-two factors (one alone would leave the fp32 range)
        const int sa = sh >> 1, sb = sh - sa;
        const float fa = pow2f(sa), fb = pow2f(sb);
        packed[0] = pack_mantissas4((x[0] * fa) * fb, (x[1] * fa) * fb, (x[2] * fa) * fb, (x[3] * fa) * fb);
        packed[1] = pack_mantissas4((x[4] * fa) * fb, (x[5] * fa) * fb, (x[6] * fa) * fb, (x[7] * fa) * fb);
    }
    return E;
}

}  // namespace bfp16
