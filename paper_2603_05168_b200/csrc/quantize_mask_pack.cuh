// Part 1 of the path: absmean ternary quantisation (Eq. 1), 2:4 magnitude mask from the master
// weights (Eq. 2), W_eff = W_q (.) M (Eq. 3), compressed value + metadata layout.
//
// gamma needs the whole matrix before any element can be rounded, so there are two passes:
//
//   pass 1  absmean_partials_kernel   sum|W| in fp64, fixed grid, one partial per CTA
//                                     (fixed assignment of elements to threads and a fixed
//                                     reduction tree -> the same bits on every run)
//   pass 2  mask_pack_kernel          every CTA re-reduces the partials in the same fixed order
//                                     (no atomics, no counter, no third launch), derives the
//                                     scale, then streams W once more: top-2-of-4, ternarise,
//                                     write vals / meta (/ dense W_q / flip count).
//                                     Pass 2 walks the matrix backwards, so what pass 1 read
//                                     last -- still resident in the 126 MB L2 -- is read first.
//
// Both passes are HBM-bound streaming kernels: 16 B loads per lane, a warp instruction covers
// 512 contiguous bytes; a warp store covers one whole 64 B (vals), 128 B (dense W_q) or 16 B
// (metadata) row of an operand tile (tiled layouts, see layouts.cuh).
//
// Ternarisation without a per-element division: W_q = sign(w) * [ fl(|w| / scale) > 0.5 ]
// (round-half-even sends exactly 0.5 to 0, everything above to >= 1, the clamp caps at 1).
// Correctly rounded division is monotone in |w|, so there is one fp32 threshold thr with
// fl(a / scale) > 0.5  <=>  a >= thr.  thr is found once per matrix with real IEEE divisions
// and the per-element work is a compare.
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kQmpThreads = 256;
constexpr int kQmpMaxPartials = kNumSMs * 4;          // pass-1 grid upper bound
constexpr int kQmpTileFloats = kQmpThreads * 16;      // 4 float4 per thread per tile

struct QmpWorkspace {            // layout of the caller's workspace
    double partial[kQmpMaxPartials];
};

// ------------------------------------------------------------------------------------------------
// pass 1
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ double block_sum_fixed(double v, double* s_warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) s_warp[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kQmpThreads / 32; ++w) t += s_warp[w];
    __syncthreads();
    return t;       // identical in every thread
}

__global__ void __launch_bounds__(kQmpThreads)
absmean_partials_kernel(const float4* __restrict__ W4, size_t n4, double* __restrict__ partial,
                        unsigned long long* __restrict__ flip_bits) {
    __shared__ double s_warp[kQmpThreads / 32];
    const size_t stride = static_cast<size_t>(gridDim.x) * kQmpThreads;
    size_t i = static_cast<size_t>(blockIdx.x) * kQmpThreads + threadIdx.x;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    // four independent 16 B loads in flight per thread
    for (; i + 3 * stride < n4; i += 4 * stride) {
        const float4 v0 = __ldg(W4 + i);
        const float4 v1 = __ldg(W4 + i + stride);
        const float4 v2 = __ldg(W4 + i + 2 * stride);
        const float4 v3 = __ldg(W4 + i + 3 * stride);
        a0 += (double)fabsf(v0.x); a1 += (double)fabsf(v0.y); a2 += (double)fabsf(v0.z); a3 += (double)fabsf(v0.w);
        a0 += (double)fabsf(v1.x); a1 += (double)fabsf(v1.y); a2 += (double)fabsf(v1.z); a3 += (double)fabsf(v1.w);
        a0 += (double)fabsf(v2.x); a1 += (double)fabsf(v2.y); a2 += (double)fabsf(v2.z); a3 += (double)fabsf(v2.w);
        a0 += (double)fabsf(v3.x); a1 += (double)fabsf(v3.y); a2 += (double)fabsf(v3.z); a3 += (double)fabsf(v3.w);
    }
    for (; i < n4; i += stride) {
        const float4 v0 = __ldg(W4 + i);
        a0 += (double)fabsf(v0.x); a1 += (double)fabsf(v0.y); a2 += (double)fabsf(v0.z); a3 += (double)fabsf(v0.w);
    }
    const double t = block_sum_fixed((a0 + a1) + (a2 + a3), s_warp);
    if (threadIdx.x == 0) {
        partial[blockIdx.x] = t;
        if (blockIdx.x == 0 && flip_bits != nullptr) *flip_bits = 0ull;   // pass 2 accumulates
    }
}

// ------------------------------------------------------------------------------------------------
// pass 2
// ------------------------------------------------------------------------------------------------
// Smallest fp32 a with fl(a / scale) > 0.5, searched around 0.5 * scale with IEEE divisions.
__device__ __forceinline__ float ternary_threshold(float scale) {
    float a = 0.5f * scale;
    for (int it = 0; it < 8 && __fdiv_rn(a, scale) > 0.5f; ++it) a = __uint_as_float(__float_as_uint(a) - 1u);
    for (int it = 0; it < 16 && !(__fdiv_rn(a, scale) > 0.5f); ++it) a = __uint_as_float(__float_as_uint(a) + 1u);
    return a;
}

// One 2:4 group: returns nibble | q-bytes.  Ranking on |w| of the fp32 master weights; on equal
// magnitudes the lower column wins.
struct GroupResult {
    uint32_t nibble;     // i0 | i1 << 2
    uint32_t vals16;     // two int8 (kept values, low byte = column i0)
    uint32_t dense32;    // four int8 (unmasked W_q)
};

__device__ __forceinline__ GroupResult process_group(const float4 w, float thr) {
    const float a0 = fabsf(w.x), a1 = fabsf(w.y), a2 = fabsf(w.z), a3 = fabsf(w.w);
    // rank_j = number of entries that beat entry j; entry i beats j>i iff a_i >= a_j
    const int c01 = a0 >= a1, c02 = a0 >= a2, c03 = a0 >= a3;
    const int c12 = a1 >= a2, c13 = a1 >= a3, c23 = a2 >= a3;
    const int r0 = (1 - c01) + (1 - c02) + (1 - c03);
    const int r1 = c01 + (1 - c12) + (1 - c13);
    const int r2 = c02 + c12 + (1 - c23);
    const int r3 = c03 + c13 + c23;
    const uint32_t keep = (r0 < 2 ? 1u : 0u) | (r1 < 2 ? 2u : 0u) | (r2 < 2 ? 4u : 0u) | (r3 < 2 ? 8u : 0u);
    // exactly two bits set: lowest and highest set bit
    const uint32_t i0 = __ffs(keep) - 1;
    const uint32_t i1 = 31 - __clz(keep);
    // ternary codes as bytes: +1 -> 0x01, -1 -> 0xFF, 0 -> 0x00
    const uint32_t q0 = a0 >= thr ? (w.x < 0.0f ? 0xFFu : 0x01u) : 0u;
    const uint32_t q1 = a1 >= thr ? (w.y < 0.0f ? 0xFFu : 0x01u) : 0u;
    const uint32_t q2 = a2 >= thr ? (w.z < 0.0f ? 0xFFu : 0x01u) : 0u;
    const uint32_t q3 = a3 >= thr ? (w.w < 0.0f ? 0xFFu : 0x01u) : 0u;
    GroupResult r;
    r.dense32 = q0 | (q1 << 8) | (q2 << 16) | (q3 << 24);
    r.nibble = i0 | (i1 << 2);
    r.vals16 = ((r.dense32 >> (8 * i0)) & 0xFFu) | (((r.dense32 >> (8 * i1)) & 0xFFu) << 8);
    return r;
}

__device__ __forceinline__ uint32_t nibble_to_mask(uint32_t nib) {
    return (1u << (nib & 3u)) | (1u << ((nib >> 2) & 3u));
}

template <bool WRITE_DENSE, bool COUNT_FLIPS>
__global__ void __launch_bounds__(kQmpThreads)
mask_pack_kernel(const float4* __restrict__ W4, size_t num_tiles, uint32_t KB,
                 double count, const double* __restrict__ partial, int num_partials,
                 uint16_t* __restrict__ vals, uint8_t* meta,
                 float* __restrict__ w_scale, uint32_t* __restrict__ dense_q,
                 const uint8_t* prev_meta, unsigned long long* __restrict__ flip_bits) {
    __shared__ double s_warp[kQmpThreads / 32];
    __shared__ float s_thr;

    // Fixed-order reduction of the pass-1 partials: thread j adds partial[j], partial[j + 256],
    // ... then the block tree; every CTA gets the same bits.
    double v = 0.0;
    for (int j = threadIdx.x; j < num_partials; j += kQmpThreads) v += partial[j];
    const double S = block_sum_fixed(v, s_warp);
    const float gamma = static_cast<float>(S / count);
    const float scale = fmaxf(gamma, kEps);
    if (threadIdx.x == 0) {
        s_thr = ternary_threshold(scale);
        if (blockIdx.x == 0) *w_scale = scale;
    }
    __syncthreads();
    const float thr = s_thr;

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    unsigned int flips = 0;

    // One warp iteration = 32 consecutive groups = one (row, 128-column block) unit; unit index
    // u = n * KB + kb.  Outputs go to the tiled layouts of layouts.cuh.
    for (size_t it = blockIdx.x; it < num_tiles; it += gridDim.x) {
        const size_t tile = num_tiles - 1 - it;                       // backwards: L2-warm first
        const size_t g_base = tile * (kQmpTileFloats / 4) + static_cast<size_t>(warp) * 128;
        const uint32_t u_base = static_cast<uint32_t>(tile * 32 + static_cast<size_t>(warp) * 4);
        uint32_t n_cur = u_base / KB;
        uint32_t kb_cur = u_base - n_cur * KB;
        float4 w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = __ldg(W4 + g_base + j * 32 + lane);
        size_t tile_idx[4];           // (n/128)*KB + kb
        uint32_t row_in_tile[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            tile_idx[j] = static_cast<size_t>(n_cur >> 7) * KB + kb_cur;
            row_in_tile[j] = n_cur & 127u;
            if (++kb_cur == KB) { kb_cur = 0; ++n_cur; }
        }
        uint32_t prev[4];
        if constexpr (COUNT_FLIPS) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                prev[j] = (lane & 1) ? 0u : prev_meta[(tile_idx[j] << 11) + (row_in_tile[j] << 4) + (lane >> 1)];
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const GroupResult r = process_group(w[j], thr);
            const uint32_t rr = row_in_tile[j];
            // compressed columns 2*lane, 2*lane+1 of this 64 B tile row
            vals[((tile_idx[j] << 13) + vals_in_tile(rr, 2u * lane)) >> 1] = static_cast<uint16_t>(r.vals16);
            if constexpr (WRITE_DENSE) dense_q[((tile_idx[j] << 14) + sw128_in_tile(rr, 4u * lane)) >> 2] = r.dense32;
            const uint32_t hi = __shfl_down_sync(0xFFFFFFFFu, r.nibble, 1);
            if ((lane & 1) == 0) {
                const uint32_t byte = r.nibble | (hi << 4);
                if constexpr (COUNT_FLIPS) {
                    flips += __popc(nibble_to_mask(byte & 15u) ^ nibble_to_mask(prev[j] & 15u)) +
                             __popc(nibble_to_mask(byte >> 4) ^ nibble_to_mask((prev[j] >> 4) & 15u));
                }
                meta[(tile_idx[j] << 11) + (rr << 4) + (lane >> 1)] = static_cast<uint8_t>(byte);
            }
        }
    }

    if constexpr (COUNT_FLIPS) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) flips += __shfl_xor_sync(0xFFFFFFFFu, flips, o);
        __shared__ unsigned int s_flips[kQmpThreads / 32];
        if (lane == 0) s_flips[warp] = flips;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long t = 0;
#pragma unroll
            for (int w2 = 0; w2 < kQmpThreads / 32; ++w2) t += s_flips[w2];
            if (t) atomicAdd(flip_bits, t);
        }
    }
}

inline int qmp_num_partials(size_t n4) {
    const size_t per_cta = static_cast<size_t>(kQmpThreads) * 4;
    size_t want = (n4 + per_cta - 1) / per_cta;
    if (want < 1) want = 1;
    if (want > static_cast<size_t>(kQmpMaxPartials)) want = kQmpMaxPartials;
    return static_cast<int>(want);
}

inline sbn_status launch_quantize_mask_pack(const float* W, int N, int K, int8_t* vals,
                                            uint8_t* meta, float* w_scale, int8_t* dense_q,
                                            const uint8_t* prev_meta,
                                            unsigned long long* flip_bits, double* partial,
                                            cudaStream_t stream) {
    const size_t count = static_cast<size_t>(N) * K;
    const size_t n4 = count / 4;
    const int P = qmp_num_partials(n4);
    absmean_partials_kernel<<<P, kQmpThreads, 0, stream>>>(
        reinterpret_cast<const float4*>(W), n4, partial, prev_meta ? flip_bits : nullptr);
    ++g_launch_count;

    const size_t num_tiles = count / kQmpTileFloats;
    size_t grid = num_tiles < static_cast<size_t>(kNumSMs * 8) ? num_tiles : kNumSMs * 8;
    const float4* W4 = reinterpret_cast<const float4*>(W);
    uint16_t* v16 = reinterpret_cast<uint16_t*>(vals);
    uint32_t* d32 = reinterpret_cast<uint32_t*>(dense_q);
    const double cnt = static_cast<double>(count);
#define SBN_QMP_LAUNCH(D, F)                                                                   \
    mask_pack_kernel<D, F><<<static_cast<unsigned>(grid), kQmpThreads, 0, stream>>>(           \
        W4, num_tiles, static_cast<uint32_t>(K / 128), cnt, partial, P, v16, meta, w_scale, d32, prev_meta, flip_bits)
    if (dense_q && prev_meta) SBN_QMP_LAUNCH(true, true);
    else if (dense_q) SBN_QMP_LAUNCH(true, false);
    else if (prev_meta) SBN_QMP_LAUNCH(false, true);
    else SBN_QMP_LAUNCH(false, false);
#undef SBN_QMP_LAUNCH
    ++g_launch_count;
    return cudaGetLastError() == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
