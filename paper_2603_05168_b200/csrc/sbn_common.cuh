// Shared declarations of the libsbn translation unit (device status word, small helpers).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <atomic>
#include <utility>

#include "sbn.h"

namespace sbn {

constexpr int kNumSMs = 148;          // B200: 2 dies x 74 SMs
constexpr float kEps = 1e-5f;         // Algorithm 2's clamp for both scales

// Device status word: 0 = fine, otherwise an sbn_status written by a kernel whose bounded wait
// ran out.  Read and cleared by sbn_check_status.
__device__ int g_device_status = 0;

// Limit of every bounded device-side wait, in ns (default 2 s).  Only the slow path of a wait reads it
// (after the first polls have failed); sbn_set_wait_test shortens it so that a test can make a wait
// run out without anything hanging.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
__device__ unsigned long long g_wait_limit_ns = kWaitLimitNs;

// Host state of sbn_set_wait_test: non-zero makes the producers of the GEMM kernels issue no loads and
// the last CTA of the pack kernel withhold its partial sum -- the consumers' waits then run out.
static int g_test_break_waits = 0;
// Host state of sbn_set_gemm_probe (timing experiments on the CTA-pair kernel; 0 = normal operation).
static int g_gemm_probe = 0;

// Host-side count of kernel launches made by the library.
static std::atomic<unsigned long long> g_launch_count{0ull};

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialisation attribute and starts with
//     pdl_launch_dependents();  <set-up that touches no global memory>;  pdl_wait();
// pdl_wait returns once the preceding kernel of the stream has completed and its writes are
// visible, so everything after it is ordered exactly as in a plain stream; what is gained is
// that the CTAs of the next kernel become resident (and do their set-up) on SMs the previous
// kernel has already left, instead of after a full launch round trip.  The signal comes first, so
// in a chain of short kernels (quantiser, GEMM, quantiser, GEMM, ...) a kernel is resident while
// the one TWO places ahead still runs: its own wait keeps it correct, and a GEMM uses the time to
// fetch weights.  All kernels here are
// persistent with every CTA resident from the start, so an early dependent only ever takes
// resources nobody else is waiting for.  SBN_DISABLE_PDL=1 in the environment turns the
// attribute off (the two instructions are then no-ops).
// One exception in each direction, which belong together: the few-token GEMM kernel fetches its
// first stages of WEIGHTS before pdl_wait (they do not depend on the kernel right before it in a
// decode loop, and their latency is most of that kernel's time), and in return the kernels that
// WRITE packed weights (quantize_mask_pack) never call pdl_launch_dependents.  Without that signal
// a successor starts only after the writer has completed and flushed, so any kernel that is
// running -- and everything it may have launched early -- comes after every weight producer.
// Weights written by copies or by kernels of other libraries are ordered the same way (they give no
// early signal); a caller's own kernel that writes vals / meta must not give one either.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

inline bool pdl_enabled() {
    static const bool on = [] {
        const char* e = getenv("SBN_DISABLE_PDL");
        return !(e && e[0] == '1');
    }();
    return on;
}

// Opt-in to more than 48 KB of dynamic shared memory.  The attribute is per device, so it is set once
// per (kernel, device); the record is a bit mask per kernel instantiation (devices beyond 63 simply
// set it on every launch).  Safe to call from several host threads.
template <auto Kernel>
inline bool ensure_dynamic_smem(int bytes) {
    static std::atomic<unsigned long long> done{0ull};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return true;
    if (cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
    return true;
}

// SMs of the current device (cached per device; kNumSMs if the query fails).
inline int device_sm_count() {
    static std::atomic<int> cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kNumSMs;
    int n = cached[dev].load(std::memory_order_acquire);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = kNumSMs;
        cached[dev].store(n, std::memory_order_release);
    }
    return n;
}

// `cluster` > 1 launches the grid as clusters of that many consecutive CTAs (runtime cluster size).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                         unsigned cluster, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args&&... args) {
    return launch_kernel_cluster(kernel, grid, block, smem, stream, 0u, std::forward<Args>(args)...);
}

// Ask the L2 to fetch [p, p + bytes) (a multiple of 16 B) -- issued by one thread, no destination.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

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
