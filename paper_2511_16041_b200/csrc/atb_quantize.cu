// atb_quantize_bfp16: fp32 -> BFP16 planes (format of Section 2.4).  HBM-bound streaming kernel:
// 4 B read and 1.125 B written per element.
//
// One CTA of 256 threads quantises a tile of 32 rows x 256 columns (32 blocks of 8 per row).
// Warp w owns rows 4w..4w+3; lane l owns block l of each of its rows, so a warp reads 1 KB of
// one row and writes 256 contiguous mantissa bytes.  The 8 block exponents of a (row, 64-column
// panel) pair are contiguous in the exponent plane and rows are adjacent, so they are staged in
// shared memory and written by 128 threads as one 256-byte run per panel.
#include <cuda_runtime.h>

#include <cstdint>

#include "atb_internal.h"
#include "bfp16_block.cuh"

namespace {

constexpr int kTileRows = 32;
constexpr int kTileBlocks = 32;   // blocks of 8 columns per tile row
constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
quantize_bfp16_kernel(const float* __restrict__ A, int64_t M, int64_t K, int64_t lda,
                      int8_t* __restrict__ mant, uint8_t* __restrict__ exp_plane, int64_t M_pad) {
    __shared__ __align__(16) uint8_t s_exp[4][kTileRows][8];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t KB = K >> 3;
    const int64_t kb = static_cast<int64_t>(blockIdx.x) * kTileBlocks + lane;
    const int64_t m0 = static_cast<int64_t>(blockIdx.y) * kTileRows;
    const bool kb_ok = kb < KB;

    float4 lo[4], hi[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + warp * 4 + i;
        if (kb_ok && m < M) {
            const float4* p = reinterpret_cast<const float4*>(A + m * lda + kb * 8);
            lo[i] = __ldg(p);
            hi[i] = __ldg(p + 1);
        } else {
            lo[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            hi[i] = lo[i];
        }
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + warp * 4 + i;
        const float x[8] = {lo[i].x, lo[i].y, lo[i].z, lo[i].w, hi[i].x, hi[i].y, hi[i].z, hi[i].w};
        uint32_t packed[2];
        const int E = bfp16::quantize_block8(x, packed);
        if (kb_ok && m < M)
            *reinterpret_cast<uint2*>(mant + m * K + kb * 8) = make_uint2(packed[0], packed[1]);
        s_exp[lane >> 3][warp * 4 + i][lane & 7] = (kb_ok && m < M) ? static_cast<uint8_t>(E) : 0;
    }
    __syncthreads();

    if (threadIdx.x < 4 * kTileRows) {
        const int panel = threadIdx.x >> 5, row = threadIdx.x & 31;
        const int64_t p = static_cast<int64_t>(blockIdx.x) * 4 + panel;
        if (p < (K + 63) / 64) {
            const uint64_t v = *reinterpret_cast<const uint64_t*>(&s_exp[panel][row][0]);
            *reinterpret_cast<uint64_t*>(exp_plane + (p * M_pad + m0 + row) * 8) = v;
        }
    }
}

}  // namespace

extern "C" atb_status_t atb_quantize_bfp16(const float* A_dev, int64_t M, int64_t K, int64_t lda,
                                           int8_t* mant_dev, uint8_t* exp_dev, void* stream) {
    atb::clear_error();
    if (M < 0 || K < 0) return atb::fail(ATB_ERR_BAD_SHAPE, "M=%lld, K=%lld must be >= 0", (long long)M, (long long)K);
    if (K % 8 != 0) return atb::fail(ATB_ERR_BAD_SHAPE, "K=%lld is not a multiple of the block size 8", (long long)K);
    if (M == 0 || K == 0) return ATB_OK;
    if (!A_dev || !mant_dev || !exp_dev) return atb::fail(ATB_ERR_NULL_POINTER, "A_dev, mant_dev and exp_dev must be non-NULL");
    if (lda < K || lda % 4 != 0) return atb::fail(ATB_ERR_BAD_SHAPE, "lda=%lld must be >= K and a multiple of 4", (long long)lda);
    if (!atb::aligned16(A_dev) || !atb::aligned16(mant_dev) || !atb::aligned16(exp_dev))
        return atb::fail(ATB_ERR_MISALIGNED, "A_dev, mant_dev and exp_dev must be 16-byte aligned");
    const int64_t M_pad = atb::round_up(M, 32);
    const int64_t grid_x = atb::ceil_div(K / 8, kTileBlocks), grid_y = M_pad / kTileRows;
    if (grid_y > 65535) return atb::fail(ATB_ERR_BAD_SHAPE, "M=%lld exceeds 65535*32 rows", (long long)M);
    dim3 grid(static_cast<unsigned>(grid_x), static_cast<unsigned>(grid_y));
    quantize_bfp16_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        A_dev, M, K, lda, mant_dev, exp_dev, M_pad);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return atb::fail(ATB_ERR_CUDA, "quantize launch: %s", cudaGetErrorString(e));
    return ATB_OK;
}
