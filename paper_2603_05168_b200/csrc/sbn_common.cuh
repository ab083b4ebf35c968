// Shared declarations of the libsbn translation unit (device status word, small helpers).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sbn.h"

namespace sbn {

constexpr int kNumSMs = 148;          // B200: 2 dies x 74 SMs
constexpr float kEps = 1e-5f;         // Algorithm 2's clamp for both scales

// Device status word: 0 = fine, otherwise an sbn_status written by a kernel whose bounded wait
// ran out.  Read and cleared by sbn_check_status.
__device__ int g_device_status = 0;

// Host-side count of kernel launches made by the library.
static unsigned long long g_launch_count = 0;

__device__ __forceinline__ float bf16lo_to_f32(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// fp32 -> bf16 bit pattern, round-to-nearest-even (finite inputs).
__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) {
    uint32_t u = __float_as_uint(f);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return u >> 16;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

}  // namespace sbn
