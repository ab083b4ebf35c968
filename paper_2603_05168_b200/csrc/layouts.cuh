// Operand layouts in HBM ("tiled" = stored as the exact shared-memory image of an MMA operand tile).
//
// A TMA tile load is processed row by row at roughly one box row per clock per SM, so operand
// tiles made of short rows (64 B of compressed weights, 16 B of metadata) are fetched far below
// the bandwidth the tensor core needs.  The kernels that PRODUCE the GEMM operands therefore write
// them tile by tile, already in the swizzled order the MMA descriptors expect, and the GEMM
// fetches every tile as a few 1 KB rows.  Each layout is a pure permutation of the plain
// row-major array; the formulas below are the definition (all sizes in bytes, K % 128 == 0,
// N % 128 == 0, KB = K / 128):
//
//   vals   (compressed 2:4 values, row-major [N][K/2]) -> tiles of 128 rows x 64 B, 8 KB each,
//          tile (n/128, cc/64) at ((n/128)*KB + cc/64) * 8192; inside, 64 B rows with the 16 B
//          chunk index XOR-ed by ((row/2) & 3)                          [SWIZZLE_64B image]
//   meta   (row-major [N][K/8]) -> tiles of 128 rows x 16 B, 2 KB each, tile (n/128, b/16) at
//          ((n/128)*KB + b/16) * 2048; inside, row r at r*16              [no swizzle]
//   dense_q (row-major [N][K]) -> tiles of 128 rows x 128 B, 16 KB each, tile (n/128, k/128) at
//          ((n/128)*KB + k/128) * 16384; inside, 8-row atoms of 1 KB, 128 B rows with the 16 B
//          chunk index XOR-ed by (row & 7)                              [SWIZZLE_128B image]
//   xq     (row-major [T][K]) -> atoms of 8 tokens x 128 B, 1 KB each, atom (k/128, t/8) at
//          ((k/128)*TB8 + t/8) * 1024 with TB8 = 2*ceil(T/16); inside as for dense_q
//          [SWIZZLE_128B image]; the buffer holds KB*TB8 atoms (tokens padded to a multiple of 16;
//          padding rows are never read for a stored output)
#pragma once

#include <stddef.h>
#include <stdint.h>

namespace sbn {

__host__ __device__ inline size_t xq_tb8(int T) { return 2 * static_cast<size_t>((T + 15) / 16); }
__host__ __device__ inline size_t xq_tiled_bytes(int T, int K) { return xq_tb8(T) * static_cast<size_t>(K / 128) * 1024; }

// byte offset inside an 8 KB vals tile of (row r, compressed byte column c in 0..63)
__host__ __device__ inline uint32_t vals_in_tile(uint32_t r, uint32_t c) {
    return (r << 6) + ((((c >> 4) ^ ((r >> 1) & 3u))) << 4) + (c & 15u);
}
// byte offset inside a 16 KB dense tile / inside a 1 KB-atom stack of (row r, byte column c in 0..127)
__host__ __device__ inline uint32_t sw128_in_tile(uint32_t r, uint32_t c) {
    return ((r >> 3) << 10) + ((r & 7u) << 7) + ((((c >> 4) ^ (r & 7u))) << 4) + (c & 15u);
}

}  // namespace sbn
