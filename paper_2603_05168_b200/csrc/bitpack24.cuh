// Packed storage of the kept 2:4 values for the weight-bound few-token regime.
//
// The int8-held form spends 5 bits per weight (two value bytes + one metadata nibble per group of
// four).  A kept value is ternary, so two bits hold it (t = v + 1 in {0, 1, 2}); the two values of a
// group share a nibble, t0 | t1 << 2, even groups in the low nibble of their byte.  With the
// metadata left as it is that makes 2 bits per weight, and expanding costs three ALU instructions
// per group and no table.  (A denser 6-bit code per group -- 54 states, 1.5 bits per weight -- was
// built first: its table look-ups made the GEMM slower than with int8-held weights.)
// Layout: vals2 is [N][K/8] bytes stored tile by tile like the metadata: 2 KB per (128 rows,
// 128 columns) block at ((n / 128) * K/128 + k / 128) * 2048, row r of the block at r * 16.
// pack_vals2_kernel converts the tiled vals (once, when weights are loaded); the few-token GEMM of
// gemm_packed_cluster_tcgen05.cuh expands tiles back into its shared-memory operand image.
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kVals2TileBytes = 128 * 16;

// 16 value bytes (8 groups) -> 8 nibbles in one word
__device__ __forceinline__ uint32_t pack_vals2_chunk(const uint4 v) {
    const uint32_t t[4] = {__vadd4(v.x, 0x01010101u), __vadd4(v.y, 0x01010101u), __vadd4(v.z, 0x01010101u), __vadd4(v.w, 0x01010101u)};
    uint32_t out = 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // bytes t0 t1 t0' t1' (each 0..2) -> t0 | t1 << 2 | t0' << 4 | t1' << 6
        const uint32_t x = t[i];
        const uint32_t b = (x & 3u) | ((x >> 6) & 0xCu) | ((x >> 12) & 0x30u) | ((x >> 18) & 0xC0u);
        out |= b << (8 * i);
    }
    return out;
}

// Thread (row, 16 B chunk): a CTA of 128 threads converts 32 rows of a tile per step.
__global__ void __launch_bounds__(128)
pack_vals2_kernel(const uint8_t* __restrict__ vals, uint8_t* __restrict__ vals2, int tiles) {
    pdl_wait();                            // writes weights: no early signal to the next kernel
    const uint32_t c = threadIdx.x & 3u;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t r = (threadIdx.x >> 2) + 32u * i;
            const uint4 v = *reinterpret_cast<const uint4*>(vals + static_cast<size_t>(tile) * 8192 + r * 64 + ((c ^ ((r >> 1) & 3u)) << 4));
            *reinterpret_cast<uint32_t*>(vals2 + static_cast<size_t>(tile) * kVals2TileBytes + r * 16 + 4 * c) = pack_vals2_chunk(v);
        }
    }
}

inline sbn_status launch_pack_vals2(const int8_t* vals, int N, int K, uint8_t* vals2, cudaStream_t stream) {
    const int tiles = (N / 128) * (K / 128);
    const int grid = std::min(tiles, 8 * device_sm_count());
    const cudaError_t err = launch_kernel(pack_vals2_kernel, dim3(grid), dim3(128), 0, stream,
                                          reinterpret_cast<const uint8_t*>(vals), vals2, tiles);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
