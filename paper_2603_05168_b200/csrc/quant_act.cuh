// Per-token absmax int8 activation quantiser (Sec. 2.1; Algorithm 2, forward step 1).
//
//   a = max_k |x|, d = max(a, 1e-5), s_x = 127 / d,
//   xq = clamp(rint(x * s_x), -128, 127),  a_scale = d / 127
//
// HBM-bound: 2 B read + 1 B written per element.  A group of G threads owns one token row and
// keeps it in registers between the max and the rounding, so x is read from memory once.
// Loads are 16 B (8 bf16) per lane, stores 8 B (8 int8) per lane, both fully coalesced.
// xq is written in the tiled layout of layouts.cuh (8-token x 128 B swizzled atoms), which moves
// 16 B chunks around inside a 128 B line but keeps every warp store a set of whole lines.
#pragma once

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kActThreads = 256;

// |x| of non-negative bf16 bit patterns orders like unsigned integers, so the row maximum is
// taken on packed halfwords: clear the two sign bits, then a per-halfword unsigned max.
__device__ __forceinline__ uint32_t absmax8_packed(const uint4& v, uint32_t m) {
    constexpr uint32_t kAbs = 0x7FFF7FFFu;
    m = __vmaxu2(m, __vmaxu2(__vmaxu2(v.x & kAbs, v.y & kAbs), __vmaxu2(v.z & kAbs, v.w & kAbs)));
    return m;
}
__device__ __forceinline__ float packed_max_to_f32(uint32_t m) {
    return __uint_as_float(max(m >> 16, m & 0xFFFFu) << 16);
}
__device__ __forceinline__ float absmax8(const uint4& v) { return packed_max_to_f32(absmax8_packed(v, 0u)); }

// round(x * s_x) for two values, saturated to int8 and packed: (sat8(a) << 8 | sat8(b)) | c << 16.
// The saturation is Algorithm 2's clamp(-128, 127).
__device__ __forceinline__ uint32_t pack_sat_s8x2(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int quant1(float x, float s_x) {
    return __float2int_rn(__fmul_rn(x, s_x));      // one fp32 multiply, then half-to-even
}
// four consecutive bf16 (two words) -> four int8 codes in one word, lowest column in the low byte
__device__ __forceinline__ uint32_t quant_pair2(uint32_t a, uint32_t b, float s_x) {
    const uint32_t hi = pack_sat_s8x2(quant1(bf16hi_to_f32(b), s_x), quant1(bf16lo_to_f32(b), s_x), 0u);
    return pack_sat_s8x2(quant1(bf16hi_to_f32(a), s_x), quant1(bf16lo_to_f32(a), s_x), hi);
}

// Index (in 8-byte units) of the 8 int8 codes of token `t`, vector `idx` (columns 8*idx .. 8*idx+7).
__device__ __forceinline__ size_t xq_tiled_u2_index(int t, int idx, size_t tb8) {
    const uint32_t kb = static_cast<uint32_t>(idx) >> 4;
    const uint32_t chunk = (static_cast<uint32_t>(idx) & 15u) >> 1;
    const uint32_t half = static_cast<uint32_t>(idx) & 1u;
    const uint32_t r = static_cast<uint32_t>(t) & 7u;
    const size_t atom = static_cast<size_t>(kb) * tb8 + (static_cast<uint32_t>(t) >> 3);
    return (atom << 7) + (r << 4) + ((chunk ^ r) << 1) + half;
}

// The 6:8 pattern runs on the 2:4 tensor cores over activations expanded from K to K' = 3K/2
// columns (quantize_mask_pack68.cuh): every group of 8 codes q0..q7 becomes the three windows
// q0..q3 | q2..q5 | q4..q7, i.e. K' column 12 g + 4 w + s holds column 8 g + 2 w + s.  A lane's
// 8 codes become 12 bytes; the 48 bytes of four adjacent lanes (a quad) are three whole 16-byte
// chunks of the tiled [T][K'] layout, which lanes 0..2 of the quad store after one exchange.
// Index (in 16-byte units) of chunk c (0..2) of the quad that starts at group idx4 (a multiple of 4)
// of token t.
__device__ __forceinline__ size_t xq68_tiled_u4_index(int t, int idx4, int c, size_t tb8) {
    const uint32_t kp = 12u * static_cast<uint32_t>(idx4) + 16u * static_cast<uint32_t>(c);   // K' byte column
    const uint32_t kb = kp >> 7;
    const uint32_t chunk = (kp & 127u) >> 4;
    const uint32_t r = static_cast<uint32_t>(t) & 7u;
    const size_t atom = static_cast<size_t>(kb) * tb8 + (static_cast<uint32_t>(t) >> 3);
    return (atom << 6) + (r << 3) + (chunk ^ r);
}
// Stores the 8 codes (o.x = q0..q3, o.y = q4..q7) of group idx of token t: plain, or expanded.
// Expanded: must be reached by all 32 lanes of a warp together (idx consecutive over the lanes).
template <bool EXPAND68>
__device__ __forceinline__ void store_codes8(uint2* __restrict__ xq, int t, int idx, size_t tb8, const uint2 o) {
    if constexpr (EXPAND68) {
        const uint32_t mid = __byte_perm(o.x, o.y, 0x5432);                          // q2 q3 q4 q5
        const uint32_t na = __shfl_down_sync(0xFFFFFFFFu, o.x, 1);
        const uint32_t nm = __shfl_down_sync(0xFFFFFFFFu, mid, 1);
        const uint32_t nc = __shfl_down_sync(0xFFFFFFFFu, o.y, 1);
        const int j = idx & 3;
        // the quad's 12 words are a m c | a m c | a m c | a m c; lane j stores words 4j .. 4j+3
        uint4 v;
        v.x = j == 0 ? o.x : (j == 1 ? mid : o.y);
        v.y = j == 0 ? mid : (j == 1 ? o.y : na);
        v.z = j == 0 ? o.y : (j == 1 ? na : nm);
        v.w = j == 0 ? na : (j == 1 ? nm : nc);
        if (j < 3) reinterpret_cast<uint4*>(xq)[xq68_tiled_u4_index(t, idx & ~3, j, tb8)] = v;
    } else {
        xq[xq_tiled_u2_index(t, idx, tb8)] = o;
    }
}

// G threads per token row, VPT 16-byte vectors per thread (G * VPT >= K / 8).  Persistent CTAs:
// every row group walks over rows with a grid-sized stride and loads its NEXT row while it reduces,
// rounds and stores the current one, so each SM always has loads in flight (a non-pipelined
// version of this kernel was latency-bound at a third of the HBM rate).
template <int G, int VPT, bool EXPAND68 = false>
__global__ void __launch_bounds__(kActThreads, (VPT <= 4) ? 3 : 2)
quant_act_kernel(const uint4* __restrict__ x, int T, int nvec, uint2* __restrict__ xq,
                 float* __restrict__ a_scale) {
    constexpr int ROWS = kActThreads / G;
    constexpr int WARPS_PER_ROW = (G + 31) / 32;
    __shared__ float s_max[2][kActThreads / 32];

    const int r = threadIdx.x / G;
    const int g = threadIdx.x % G;
    const int row_stride = gridDim.x * ROWS;
    const size_t tb8 = xq_tb8(T);
    const int iters = (T + row_stride - 1) / row_stride;        // same for every thread of the CTA

    pdl_launch_dependents();             // the next kernel may become resident (and fetch weights) right away
    pdl_wait();

    uint4 cur[VPT], nxt[VPT];
    int row = blockIdx.x * ROWS + r;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = g + i * G;
        cur[i] = (row < T && idx < nvec) ? __ldcs(x + static_cast<size_t>(row) * nvec + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
    for (int it = 0; it < iters; ++it, row += row_stride) {
        const int row_n = row + row_stride;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = g + i * G;
            nxt[i] = (row_n < T && idx < nvec) ? __ldcs(x + static_cast<size_t>(row_n) * nvec + idx) : make_uint4(0u, 0u, 0u, 0u);
        }
        uint32_t pm = 0u;
#pragma unroll
        for (int i = 0; i < VPT; ++i) pm = absmax8_packed(cur[i], pm);
        // bit patterns of non-negative floats order like integers: one redux instruction per warp
        float amax = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, max(pm >> 16, pm & 0xFFFFu)) << 16);
        if constexpr (WARPS_PER_ROW > 1) {
            const int warp = threadIdx.x >> 5;
            float* sm = s_max[it & 1];                               // double buffered: one barrier per row
            if ((threadIdx.x & 31) == 0) sm[warp] = amax;
            __syncthreads();
            const int w0 = (r * G) >> 5;
            float m = sm[w0];
#pragma unroll
            for (int w = 1; w < WARPS_PER_ROW; ++w) m = fmaxf(m, sm[w0 + w]);
            amax = m;
        }
        if (row < T) {
            const float d = fmaxf(amax, kEps);
            const float s_x = __fdiv_rn(127.0f, d);
            if (g == 0) a_scale[row] = __fdiv_rn(d, 127.0f);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int idx = g + i * G;
                if (idx < nvec) {
                    uint2 o;
                    o.x = quant_pair2(cur[i].x, cur[i].y, s_x);
                    o.y = quant_pair2(cur[i].z, cur[i].w, s_x);
                    store_codes8<EXPAND68>(xq, row, idx, tb8, o);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) cur[i] = nxt[i];
    }
}

// Rows too long for the register-resident kernel (K > 16384): one CTA per row, two passes over
// the row (the second one served by L1/L2).
template <bool EXPAND68 = false>
__global__ void __launch_bounds__(kActThreads)
quant_act_long_row_kernel(const uint4* __restrict__ x, int T, int nvec, uint2* __restrict__ xq,
                          float* __restrict__ a_scale) {
    __shared__ float s_max[kActThreads / 32];
    pdl_launch_dependents();             // the next kernel may become resident (and fetch weights) right away
    pdl_wait();
    const int row = blockIdx.x;
    if (row >= T) return;
    const uint4* xr = x + static_cast<size_t>(row) * nvec;
    float amax = 0.0f;
    for (int idx = threadIdx.x; idx < nvec; idx += kActThreads) amax = fmaxf(amax, absmax8(__ldg(xr + idx)));
    amax = warp_max(amax);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    float m = s_max[0];
#pragma unroll
    for (int w = 1; w < kActThreads / 32; ++w) m = fmaxf(m, s_max[w]);
    const float d = fmaxf(m, kEps);
    const float s_x = __fdiv_rn(127.0f, d);
    if (threadIdx.x == 0) a_scale[row] = __fdiv_rn(d, 127.0f);
    const size_t tb8 = xq_tb8(T);
    for (int idx = threadIdx.x; idx < nvec; idx += kActThreads) {
        const uint4 v = __ldg(xr + idx);
        uint2 o;
        o.x = quant_pair2(v.x, v.y, s_x);
        o.y = quant_pair2(v.z, v.w, s_x);
        store_codes8<EXPAND68>(xq, row, idx, tb8, o);
    }
}

template <int G, int VPT, bool EXPAND68>
static void launch_quant_act_cfg(const uint4* x, int T, int nvec, uint2* q, float* a_scale, cudaStream_t stream) {
    constexpr int rows = kActThreads / G;
    const int ctas_per_sm = (VPT <= 4) ? 3 : 2;
    int grid = (T + rows - 1) / rows;
    if (grid > kNumSMs * ctas_per_sm) grid = kNumSMs * ctas_per_sm;
    launch_kernel(quant_act_kernel<G, VPT, EXPAND68>, dim3(grid), dim3(kActThreads), 0, stream, x, T, nvec, q, a_scale);
}

template <bool EXPAND68 = false>
inline sbn_status launch_quant_act(const void* x_bf16, int T, int K, int8_t* xq, float* a_scale,
                                   cudaStream_t stream) {
    const int nvec = K / 8;
    const uint4* x = static_cast<const uint4*>(x_bf16);
    uint2* q = reinterpret_cast<uint2*>(xq);
    // smallest group that keeps <= 3 (then 4, 6, 8) vectors per thread
    if (nvec <= 32 * 2) launch_quant_act_cfg<32, 2, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 64 * 2) launch_quant_act_cfg<64, 2, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 128 * 2) launch_quant_act_cfg<128, 2, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 128 * 3) launch_quant_act_cfg<128, 3, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 256 * 2) launch_quant_act_cfg<256, 2, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 256 * 3) launch_quant_act_cfg<256, 3, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 256 * 4) launch_quant_act_cfg<256, 4, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 256 * 6) launch_quant_act_cfg<256, 6, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else if (nvec <= 256 * 8) launch_quant_act_cfg<256, 8, EXPAND68>(x, T, nvec, q, a_scale, stream);
    else launch_kernel(quant_act_long_row_kernel<EXPAND68>, dim3(T), dim3(kActThreads), 0, stream, x, T, nvec, q, a_scale);
    ++g_launch_count;
    return cudaGetLastError() == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
