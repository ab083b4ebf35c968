// The compressed 2:4 weights between the plain row-major arrays of the layout definition
// (vals [N][K/2], meta [N][K/8]: Eq. 3 stored as kept values + 2-bit indices) and the tiled order the
// GEMM kernels consume (layouts.cuh).  Both directions are pure permutations that keep every
// aligned 16-byte chunk of a row intact, so one thread moves one chunk with a 16-byte load and store.
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kCanonThreads = 256;

// TO_TILED = false: tiled -> plain;  true: plain -> tiled.  vals chunks first, then meta chunks.
template <bool TO_TILED>
__global__ void __launch_bounds__(kCanonThreads)
canonical_layout_kernel(const uint4* __restrict__ vals_in, uint4* __restrict__ vals_out,
                        const uint4* __restrict__ meta_in, uint4* __restrict__ meta_out, uint32_t N, uint32_t K) {
    // Reads (or writes) packed weights: ordered after every earlier kernel of the stream, and no early
    // start for the kernels behind it (the few-token GEMM fetches weights before its own wait).
    pdl_wait();
    const uint32_t KB = K >> 7;
    const uint64_t v_chunks = vals_in ? static_cast<uint64_t>(N) * (K >> 5) : 0ull;      // K/2 bytes per row / 16
    const uint64_t m_chunks = meta_in ? static_cast<uint64_t>(N) * (K >> 7) : 0ull;      // K/8 bytes per row / 16
    const uint64_t total = v_chunks + m_chunks;
    for (uint64_t i = static_cast<uint64_t>(blockIdx.x) * kCanonThreads + threadIdx.x; i < total;
         i += static_cast<uint64_t>(gridDim.x) * kCanonThreads) {
        if (i < v_chunks) {
            const uint32_t per_row = K >> 5;
            const uint32_t n = static_cast<uint32_t>(i / per_row), ch = static_cast<uint32_t>(i % per_row);
            const uint32_t c = ch << 4;                                       // first compressed byte column of the chunk
            const uint64_t tiled = (static_cast<uint64_t>(n >> 7) * KB + (c >> 6)) * 8192u + vals_in_tile(n & 127u, c & 63u);
            if (TO_TILED) vals_out[tiled >> 4] = vals_in[i];
            else vals_out[i] = vals_in[tiled >> 4];
        } else {
            const uint64_t j = i - v_chunks;
            const uint32_t n = static_cast<uint32_t>(j / KB), kb = static_cast<uint32_t>(j % KB);
            const uint64_t tiled = (static_cast<uint64_t>(n >> 7) * KB + kb) * 2048u + ((n & 127u) << 4);
            if (TO_TILED) meta_out[tiled >> 4] = meta_in[j];
            else meta_out[j] = meta_in[tiled >> 4];
        }
    }
}

template <bool TO_TILED>
inline sbn_status launch_canonical_layout(const void* vals_in, void* vals_out, const void* meta_in, void* meta_out,
                                          int N, int K, cudaStream_t stream) {
    const uint64_t chunks = static_cast<uint64_t>(N) * (K >> 5) + static_cast<uint64_t>(N) * (K >> 7);
    uint64_t blocks = (chunks + kCanonThreads - 1) / kCanonThreads;
    const uint64_t cap = static_cast<uint64_t>(device_sm_count()) * 8;
    if (blocks > cap) blocks = cap;
    const cudaError_t err = launch_kernel(canonical_layout_kernel<TO_TILED>, dim3(static_cast<unsigned>(blocks)), dim3(kCanonThreads), 0, stream,
                                          static_cast<const uint4*>(vals_in), static_cast<uint4*>(vals_out),
                                          static_cast<const uint4*>(meta_in), static_cast<uint4*>(meta_out),
                                          static_cast<uint32_t>(N), static_cast<uint32_t>(K));
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
