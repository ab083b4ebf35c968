// x~ = Q_a(Norm(x)) (Algorithm 1, forward), Norm read as RMSNorm with a per-channel gain g:
//
//   ms = mean_k x^2 (fp64 accumulation, one cast to fp32),  r = 1 / sqrt(ms + eps),
//   xn = (x * r) * g,   then Q_a of Sec. 2.1 on the fp32 xn:
//   a = max_k |xn|, d = max(a, 1e-5), s_x = 127 / d, xq = clamp(rint(xn * s_x), -128, 127), a_scale = d / 127
//
// One kernel, x read once: the row stays in registers (as bf16) through the three steps -- sum of
// squares, maximum of |xn|, rounding -- and xn is recomputed (two multiplies) instead of stored.
// HBM-bound like the plain quantiser: 2 B read + 1 B written per element; the normalised
// activations never exist in memory.  Same persistent-CTA row pipeline and the same tiled xq
// layout as quant_act.cuh.  The squares of bf16 values are exact in fp32 (16-bit significands); they
// are added in fp64 in a fixed order (thread-local, then a butterfly, then the warps in order).
#pragma once

#include "quant_act.cuh"

namespace sbn {

// packed fp32x2 arithmetic (two IEEE round-to-nearest operations per instruction)
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&f)[8]) {
    f[0] = bf16lo_to_f32(v.x); f[1] = bf16hi_to_f32(v.x);
    f[2] = bf16lo_to_f32(v.y); f[3] = bf16hi_to_f32(v.y);
    f[4] = bf16lo_to_f32(v.z); f[5] = bf16hi_to_f32(v.z);
    f[6] = bf16lo_to_f32(v.w); f[7] = bf16hi_to_f32(v.w);
}

// G threads per token row, VPT 16-byte vectors per thread (G * VPT >= K / 8).  The gains are copied
// to shared memory once per CTA (rows differ, channels do not).
template <int G, int VPT, bool EXPAND68 = false>
__global__ void __launch_bounds__(kActThreads, (VPT <= 4) ? 3 : 2)
norm_quant_act_kernel(const uint4* __restrict__ x, int T, int nvec, const float4* __restrict__ gain, float eps,
                      uint2* __restrict__ xq, float* __restrict__ a_scale) {
    constexpr int ROWS = kActThreads / G;
    constexpr int WARPS_PER_ROW = (G + 31) / 32;
    __shared__ double s_sum[2][kActThreads / 32];
    __shared__ float s_max[2][kActThreads / 32];

    const int r = threadIdx.x / G;
    const int g = threadIdx.x % G;
    const int warp = threadIdx.x >> 5;
    const int w0 = (r * G) >> 5;                                  // first warp of this row group
    const int row_stride = gridDim.x * ROWS;
    const size_t tb8 = xq_tb8(T);
    const int iters = (T + row_stride - 1) / row_stride;        // same for every thread of the CTA
    const bool has_gain = gain != nullptr;

    pdl_launch_dependents();             // the next kernel may become resident (and fetch weights) right away
    pdl_wait();

    extern __shared__ float4 s_gain[];                           // [nvec * 2] when a gain is given
    if (has_gain) {
        for (int i = threadIdx.x; i < 2 * nvec; i += kActThreads) s_gain[i] = __ldg(gain + i);
        __syncthreads();
    }

    uint4 cur[VPT], nxt[VPT];
    int row = blockIdx.x * ROWS + r;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = g + i * G;
        cur[i] = (row < T && idx < nvec) ? __ldg(x + static_cast<size_t>(row) * nvec + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
    for (int it = 0; it < iters; ++it, row += row_stride) {
        const int row_n = row + row_stride;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = g + i * G;
            nxt[i] = (row_n < T && idx < nvec) ? __ldg(x + static_cast<size_t>(row_n) * nvec + idx) : make_uint4(0u, 0u, 0u, 0u);
        }
        // ---- mean square
        double s4[4] = {0.0, 0.0, 0.0, 0.0};                      // four chains: the adds overlap
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            float f[8];
            bf16x8_to_f32(cur[i], f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {                                   // exact product, one rounding in the add
                const double dv = static_cast<double>(f[j]);
                s4[j & 3] = __fma_rn(dv, dv, s4[j & 3]);
            }
        }
        double ss = (s4[0] + s4[1]) + (s4[2] + s4[3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if constexpr (WARPS_PER_ROW > 1) {
            double* sm = s_sum[it & 1];
            if ((threadIdx.x & 31) == 0) sm[warp] = ss;
            __syncthreads();
            double t = 0.0;
#pragma unroll
            for (int w = 0; w < WARPS_PER_ROW; ++w) t += sm[w0 + w];
            ss = t;
        }
        const float ms = static_cast<float>(ss / static_cast<double>(nvec * 8));
        const float rinv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(ms, eps)));
        // ---- xn = (x * r) * g with packed fp32x2 multiplies, and max |xn|.  Up to four vectors per
        // thread the fp32 xn stays in registers for the rounding; longer rows recompute it.
        constexpr bool KEEP = VPT <= 4;
        const uint64_t r2 = pack_f32x2(rinv, rinv);
        uint64_t xn2[KEEP ? VPT : 1][4];
        float amax = 0.0f;
        auto normalise = [&](const uint4& v, int idx, uint64_t (&out)[4]) {
            out[0] = mul_f32x2(pack_f32x2(bf16lo_to_f32(v.x), bf16hi_to_f32(v.x)), r2);
            out[1] = mul_f32x2(pack_f32x2(bf16lo_to_f32(v.y), bf16hi_to_f32(v.y)), r2);
            out[2] = mul_f32x2(pack_f32x2(bf16lo_to_f32(v.z), bf16hi_to_f32(v.z)), r2);
            out[3] = mul_f32x2(pack_f32x2(bf16lo_to_f32(v.w), bf16hi_to_f32(v.w)), r2);
            if (has_gain && idx < nvec) {
                const float4 a = s_gain[2 * idx], b = s_gain[2 * idx + 1];
                out[0] = mul_f32x2(out[0], pack_f32x2(a.x, a.y));
                out[1] = mul_f32x2(out[1], pack_f32x2(a.z, a.w));
                out[2] = mul_f32x2(out[2], pack_f32x2(b.x, b.y));
                out[3] = mul_f32x2(out[3], pack_f32x2(b.z, b.w));
            }
        };
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            uint64_t tmp[4];
            uint64_t (&o)[4] = KEEP ? xn2[KEEP ? i : 0] : tmp;
            normalise(cur[i], g + i * G, o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float lo, hi;
                unpack_f32x2(o[j], lo, hi);
                amax = fmaxf(amax, fmaxf(fabsf(lo), fabsf(hi)));
            }
        }
        // bit patterns of non-negative floats order like integers: one redux instruction per warp
        amax = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(amax)));
        if constexpr (WARPS_PER_ROW > 1) {
            float* sm = s_max[it & 1];
            if ((threadIdx.x & 31) == 0) sm[warp] = amax;
            __syncthreads();
            float m = sm[w0];
#pragma unroll
            for (int w = 1; w < WARPS_PER_ROW; ++w) m = fmaxf(m, sm[w0 + w]);
            amax = m;
        }
        if (row < T) {
            const float d = fmaxf(amax, kEps);
            const float s_x = __fdiv_rn(127.0f, d);
            if (g == 0) a_scale[row] = __fdiv_rn(d, 127.0f);
            const uint64_t s2 = pack_f32x2(s_x, s_x);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int idx = g + i * G;
                if (idx < nvec) {
                    uint64_t tmp[4];
                    if constexpr (!KEEP) normalise(cur[i], idx, tmp);
                    const uint64_t (&o)[4] = KEEP ? xn2[KEEP ? i : 0] : tmp;
                    int q[8];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // rint(xn * s_x) for two values: multiply, then add 1.5 * 2^23 -- the adder's round-to-nearest-even
                        // IS the rounding of the method, and the integer is left in the low mantissa bits.  The
                        // adds are scalar: a packed multiply followed by a packed add came out with ONE
                        // rounding (a fused multiply-add), which breaks exact ties such as 63.5.
                        float lo, hi;
                        unpack_f32x2(mul_f32x2(o[j], s2), lo, hi);
                        q[2 * j] = static_cast<int>(__float_as_uint(__fadd_rn(lo, 12582912.0f)) - 0x4B400000u);
                        q[2 * j + 1] = static_cast<int>(__float_as_uint(__fadd_rn(hi, 12582912.0f)) - 0x4B400000u);
                    }
                    uint2 ov;                                      // lowest column in the lowest byte
                    ov.x = pack_sat_s8x2(q[1], q[0], pack_sat_s8x2(q[3], q[2], 0u));
                    ov.y = pack_sat_s8x2(q[5], q[4], pack_sat_s8x2(q[7], q[6], 0u));
                    store_codes8<EXPAND68>(xq, row, idx, tb8, ov);     // plain, or expanded for the 6:8 pattern
                }
            }
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) cur[i] = nxt[i];
    }
}

template <int G, int VPT, bool EXPAND68>
static cudaError_t launch_norm_quant_act_cfg(const uint4* x, int T, int nvec, const float4* gain, float eps, uint2* q,
                                             float* a_scale, cudaStream_t stream) {
    constexpr int rows = kActThreads / G;
    const int ctas_per_sm = (VPT <= 4) ? 3 : 2;
    int grid = (T + rows - 1) / rows;
    if (grid > kNumSMs * ctas_per_sm) grid = kNumSMs * ctas_per_sm;
    const size_t smem = gain ? static_cast<size_t>(nvec) * 32 : 0;          // K floats
    if (!ensure_dynamic_smem<norm_quant_act_kernel<G, VPT, EXPAND68>>(65536)) return cudaErrorUnknown;
    return launch_kernel(norm_quant_act_kernel<G, VPT, EXPAND68>, dim3(grid), dim3(kActThreads), smem, stream, x, T, nvec, gain, eps, q, a_scale);
}

// K up to 16384 (the register-resident row); longer rows are refused by the caller.
template <bool EXPAND68 = false>
inline sbn_status launch_norm_quant_act(const void* x_bf16, int T, int K, const float* gain, float eps, int8_t* xq,
                                        float* a_scale, cudaStream_t stream) {
    const int nvec = K / 8;
    const uint4* x = static_cast<const uint4*>(x_bf16);
    const float4* g4 = reinterpret_cast<const float4*>(gain);
    uint2* q = reinterpret_cast<uint2*>(xq);
    cudaError_t err;
    if (nvec <= 32 * 2) err = launch_norm_quant_act_cfg<32, 2, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 64 * 2) err = launch_norm_quant_act_cfg<64, 2, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 128 * 2) err = launch_norm_quant_act_cfg<128, 2, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 128 * 3) err = launch_norm_quant_act_cfg<128, 3, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 256 * 2) err = launch_norm_quant_act_cfg<256, 2, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 256 * 3) err = launch_norm_quant_act_cfg<256, 3, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 256 * 4) err = launch_norm_quant_act_cfg<256, 4, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 256 * 6) err = launch_norm_quant_act_cfg<256, 6, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else if (nvec <= 256 * 8) err = launch_norm_quant_act_cfg<256, 8, EXPAND68>(x, T, nvec, g4, eps, q, a_scale, stream);
    else return SBN_ERR_UNSUPPORTED;
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
