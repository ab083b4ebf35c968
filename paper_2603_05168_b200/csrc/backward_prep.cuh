// Operands of the backward GEMMs (dual straight-through estimator, Sec. 2.3, Eq. 5; Algorithm 2's
// backward) in bf16, as the tensor-core kernel of gemm_bf16_pair_tcgen05.cuh reads them:
//
//   dX[t][k] = sum_n dY[t][n] * w_masked[n][k]   contraction over n: A = dY [T][N] as it is (K-major),
//                                                 B = W_eff^T [K][N] (weff_t_bf16_kernel: a 128 x 128 tile
//                                                 transposed through shared memory, written as 256 B rows)
//   dW[n][k] = sum_t dY[t][n] * x_q[t][k]        contraction over t: A = dY [T][N] and B = x_q [T][K]
//                                                 (xq_bf16_kernel), both as they lie in memory; the MMA
//                                                 reads them MN-major, so nothing is transposed
//
// x_q[t][k] = bf16(x~[t][k] * a_scale[t]) are the fake-quantised activations as a bf16 training run holds
// them; W_eff is written as +-1.0 / 0.0 and its scale is applied once in the GEMM's epilogue.
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kPrepThreads = 256;
constexpr int kPrepTile = 128;
constexpr int kPrepRowBytes = kPrepTile * 2 + 16;            // bf16 row of the transposed tile, padded (keeps 16 B alignment)

__device__ __forceinline__ uint16_t bf16_bits_of(float f) { return static_cast<uint16_t>(f32_to_bf16_rne(f)); }

// Writes the transposed tile (128 rows x 128 bf16) from shared memory: row j goes to dst + j * ld
// (elements), columns [0, 128); rows >= rows_valid and 16-byte chunks beyond cols_valid are skipped.
__device__ __forceinline__ void prep_store_tile(const unsigned char* s_t, uint16_t* dst, size_t ld, int rows_valid, int cols_valid) {
    const int chunk = threadIdx.x & 15;                        // 16 B = 8 elements
    for (int j = threadIdx.x >> 4; j < kPrepTile; j += kPrepThreads / 16) {
        if (j < rows_valid && chunk * 8 < cols_valid) {
            const uint4 v = *reinterpret_cast<const uint4*>(s_t + j * kPrepRowBytes + chunk * 16);
            *reinterpret_cast<uint4*>(dst + static_cast<size_t>(j) * ld + chunk * 8) = v;
        }
    }
}

// W_eff^T [K][N] in bf16 (+-1, 0) from the compressed 2:4 form (tiled vals / meta).
__global__ void __launch_bounds__(kPrepThreads)
weff_t_bf16_kernel(const uint8_t* __restrict__ vals, const uint8_t* __restrict__ meta, int N, int K, uint16_t* __restrict__ Wt) {
    __shared__ __align__(16) unsigned char s_t[kPrepTile * kPrepRowBytes];
    pdl_wait();
    const int KB = K >> 7;
    const int kb = blockIdx.x % KB, nb = blockIdx.x / KB;
    const size_t tile = static_cast<size_t>(nb) * KB + kb;
    const int r = threadIdx.x >> 1, half = threadIdx.x & 1;    // weight row inside the tile, half of its 32 groups
    const uint2 m8 = *reinterpret_cast<const uint2*>(meta + tile * 2048 + r * 16 + half * 8);
    const uint4 v0 = *reinterpret_cast<const uint4*>(vals + tile * 8192 + vals_in_tile(r, 32u * half));
    const uint4 v1 = *reinterpret_cast<const uint4*>(vals + tile * 8192 + vals_in_tile(r, 32u * half + 16u));
    const uint32_t vw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    const uint32_t mw[2] = {m8.x, m8.y};
#pragma unroll
    for (int g = 0; g < 16; ++g) {                             // group g of this half: columns 64 half + 4 g ..
        const uint32_t nib = (mw[g >> 3] >> (4 * (g & 7))) & 15u;
        const uint32_t pair = (vw[g >> 1] >> (16 * (g & 1))) & 0xFFFFu;
        const int8_t a = static_cast<int8_t>(pair & 0xFFu), b = static_cast<int8_t>(pair >> 8);
        const uint32_t i0 = nib & 3u, i1 = nib >> 2;
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) {
            const int q = (j == i0) ? a : ((j == i1) ? b : 0);
            const uint16_t bits = q > 0 ? 0x3F80u : (q < 0 ? 0xBF80u : 0u);      // +1.0, -1.0, 0.0
            *reinterpret_cast<uint16_t*>(s_t + (64 * half + 4 * g + j) * kPrepRowBytes + r * 2) = bits;
        }
    }
    __syncthreads();
    prep_store_tile(s_t, Wt + (static_cast<size_t>(kb) * 128) * N + static_cast<size_t>(nb) * 128, static_cast<size_t>(N), kPrepTile, kPrepTile);
}

// x_q [T][K] in bf16 (token-major, as the activations themselves) from the tiled int8 activations and their
// per-token scales: the B operand of the weight-gradient GEMM when it reads MN-major operands.  A thread
// converts 16 codes (one 16 B chunk) into 32 B of output.
__global__ void __launch_bounds__(kPrepThreads)
xq_bf16_kernel(const uint8_t* __restrict__ xq, const float* __restrict__ a_scale, int T, int K, uint16_t* __restrict__ X) {
    pdl_wait();
    const size_t tb8 = xq_tb8(T);
    const int chunks_per_row = K >> 4;
    const size_t total = static_cast<size_t>(T) * chunks_per_row;
    for (size_t i = static_cast<size_t>(blockIdx.x) * kPrepThreads + threadIdx.x; i < total; i += static_cast<size_t>(gridDim.x) * kPrepThreads) {
        const int t = static_cast<int>(i / chunks_per_row), ch = static_cast<int>(i % chunks_per_row);
        const int kb = ch >> 3, c8 = ch & 7;
        const float s = __ldg(a_scale + t);
        const uint4 c = *reinterpret_cast<const uint4*>(xq + (static_cast<size_t>(kb) * tb8 + (static_cast<uint32_t>(t) >> 3)) * 1024 + (t & 7) * 128 +
                                                        ((c8 ^ (t & 7)) << 4));
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int q0 = static_cast<int8_t>((w[j >> 1] >> (16 * (j & 1))) & 0xFFu);
            const int q1 = static_cast<int8_t>((w[j >> 1] >> (16 * (j & 1) + 8)) & 0xFFu);
            o[j] = static_cast<uint32_t>(bf16_bits_of(__fmul_rn(static_cast<float>(q0), s))) |
                   (static_cast<uint32_t>(bf16_bits_of(__fmul_rn(static_cast<float>(q1), s))) << 16);
        }
        uint4* dst = reinterpret_cast<uint4*>(X + static_cast<size_t>(t) * K + static_cast<size_t>(ch) * 16);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

}  // namespace sbn
