// Bit-packed storage of the compressed 2:4 weights for the weight-bound few-token regime.
//
// The int8-held form spends 5 bits per weight (two value bytes + one metadata nibble per group of
// four).  A group has only 6 x 9 = 54 states (which two columns are kept, a ternary value each), so
// a 6-bit code per group -- 1.5 bits per weight -- carries the same information:
//     code = pair * 9 + (v0 + 1) * 3 + (v1 + 1),   pair = index of (i0, i1) in
//     (0,1) (0,2) (0,3) (1,2) (1,3) (2,3).
// Layout: one 3 KB tile per (128 rows, 128 columns) block of the matrix, tiles in the order of the
// vals tiles ((n / 128) * K/128 + k / 128); inside a tile row r owns bytes 24 r .. 24 r + 23 and the
// code of its group g (0..31) sits at bits 6 g .. 6 g + 5 of that little-endian 192-bit string.
// bitpack24_kernel converts the tiled vals + meta into this form (once, when weights are loaded);
// the few-token GEMM expands tiles back into its shared-memory operand images (see
// gemm_splitk_cluster_tcgen05.cuh).
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kPackedTileBytes = 128 * 24;

// metadata nibble (i0 | i1 << 2) -> pair index, 4 bits per entry
__device__ __forceinline__ uint32_t nibble_to_pair(uint32_t nib) {
    constexpr unsigned long long kTable = (0ull << 16) | (1ull << 32) | (2ull << 48) | (3ull << 36) | (4ull << 52) | (5ull << 56);
    return static_cast<uint32_t>(kTable >> (4u * nib)) & 15u;
}

// One thread per (row, 128-column block); a CTA of 128 threads converts one tile.
__global__ void __launch_bounds__(128)
bitpack24_kernel(const uint8_t* __restrict__ vals, const uint8_t* __restrict__ meta, uint8_t* __restrict__ packed, int tiles) {
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t r = threadIdx.x;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const uint4* vrow = reinterpret_cast<const uint4*>(vals + static_cast<size_t>(tile) * 8192 + r * 64);
        const uint4 m = *reinterpret_cast<const uint4*>(meta + static_cast<size_t>(tile) * 2048 + r * 16);
        const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
        uint32_t w[6] = {0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
        for (int c = 0; c < 4; ++c) {                              // 16 B chunk c: groups 8c .. 8c+7
            const uint4 v = vrow[c ^ ((r >> 1) & 3u)];
            const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int g = 8 * c + j;
                const uint32_t pairv = vw[j >> 1] >> (16 * (j & 1));        // two value bytes
                const int v0 = static_cast<int8_t>(pairv & 0xFFu), v1 = static_cast<int8_t>((pairv >> 8) & 0xFFu);
                const uint32_t nib = (mw[g >> 3] >> (4 * (g & 7))) & 15u;
                const uint32_t code = nibble_to_pair(nib) * 9u + static_cast<uint32_t>((v0 + 1) * 3 + (v1 + 1));
                const int bit = 6 * g;
                w[bit >> 5] |= code << (bit & 31);
                if ((bit & 31) > 26) w[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
            }
        }
        uint2* out = reinterpret_cast<uint2*>(packed + static_cast<size_t>(tile) * kPackedTileBytes + r * 24);
        out[0] = make_uint2(w[0], w[1]);
        out[1] = make_uint2(w[2], w[3]);
        out[2] = make_uint2(w[4], w[5]);
    }
}

inline sbn_status launch_bitpack24(const int8_t* vals, const uint8_t* meta, int N, int K, uint8_t* packed, cudaStream_t stream) {
    const int tiles = (N / 128) * (K / 128);
    const int grid = std::min(tiles, 8 * device_sm_count());
    const cudaError_t err = launch_kernel(bitpack24_kernel, dim3(grid), dim3(128), 0, stream,
                                          reinterpret_cast<const uint8_t*>(vals), meta, packed, tiles);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
