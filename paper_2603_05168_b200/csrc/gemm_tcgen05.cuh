// Eq. 4 on the 5th-generation tensor cores: acc[t][n] = sum_k xq[t][k] * W[n][k] (int8 x int8 ->
// int32), then y = float(acc) * (w_scale * a_scale[t]) (+ bias[n]) in the epilogue.
//
// One kernel template serves both layers:
//   SPARSE = true   W = W_eff in the compressed 2:4 layout; tcgen05.mma.sp kind::i8, logical
//                   K = 64 per instruction, metadata copied SMEM -> TMEM with tcgen05.cp
//   SPARSE = false  W = dense ternary W_q; tcgen05.mma kind::i8, K = 32 per instruction
//
// Only operand A of the MMA may be sparse, so the weights are A (M dimension = output features)
// and the activations are B (N dimension = tokens): D[n_out][token] lives in TMEM with the
// output feature on the lane axis.  The epilogue thread that owns lane n writes y[t][n] for the
// tokens in its registers; across a warp that is 32 consecutive n, i.e. one contiguous 128 B
// (fp32) or 64 B (bf16) segment per store instruction, so no transpose through shared memory is
// needed.
//
// CTA = 6 warps: warp 0 TMA producer, warp 1 MMA issuer (also owns the TMEM allocation),
// warps 2-5 epilogue (one TMEM lane quarter each).  Persistent over output tiles
// (128 features x BN tokens), static round-robin tile order, K-blocks of 128 logical columns:
//   A stage   128 rows x 64 B (sparse, SWIZZLE_64B image) or 128 rows x 128 B (dense, SWIZZLE_128B)
//   B stage   BN rows x 128 B (SWIZZLE_128B image)
//   E stage   128 rows x 16 B metadata (sparse only)
// All three are stored in HBM as these very images (layouts.cuh) and fetched as 1 KB rows.
// TMEM: ACC_STAGES accumulators of BN columns, then one 4-column metadata slot per smem stage.
//
// Every wait is bounded (wall-clock limit); a wait that runs out records SBN_ERR_TIMEOUT in the
// device status word, raises a CTA-wide abort flag and every role leaves its loop.
#pragma once

#include <cuda.h>

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kGemmThreads = 192;
constexpr int kBM = 128;                 // output features per tile (MMA M)
constexpr int kBK = 128;                 // logical K per pipeline stage
constexpr uint32_t kTmemCols = 512;
constexpr int kSmemBudget = 224 * 1024;  // of the 227 KB a CTA may use
constexpr int kEpiWarpBufBytes = 32 * 32 * 4;                 // one 32-token x 32-feature fp32 slab
constexpr int kEpiBytes = 4 * 2 * kEpiWarpBufBytes;           // 4 epilogue warps, double buffered
constexpr int kScaleBytes = 4 * 256 * 4;                      // per-token scales, one copy per epilogue warp
constexpr int kBarrierBytes = 256;

struct GemmParams {
    int T, N, K;
    int k_blocks_total;          // K / 128
    int k_splits;                // split-K factor (1 = none)
    int tb8;                     // 8-token atoms per 128-column block of the tiled xq (2*ceil(T/16))
    const float* a_scale;        // [T]
    const float* w_scale;        // [1]
    const float* bias;           // [N] or null
    void* y;                     // [T][N] fp32 or bf16
    int out_bf16;
    int32_t* acc_out;            // [T][N] or null
    int32_t* split_acc;          // [T][N] int32 scratch when k_splits > 1: zero on entry, zero again on exit
    unsigned int* split_counters;   // one per output tile, same rule
    const void* w_vals;          // the weight operand (compressed values, or the dense W_q) and its metadata
    const void* w_meta;          //   (null for dense): only used to warm the L2 before the dependency wait
    int w_tile_bytes;            // bytes of one 128 x 128 weight tile (8192 sparse, 16384 dense)
    int test_skip_loads = 0;     // diagnostics (sbn_set_wait_test): the TMA producer issues no loads, so the
                                 //   consumers' bounded waits run out and every role leaves through the abort flag
    int probe = 0;               // diagnostics (sbn_set_gemm_probe, CTA-pair kernel, timing only -- results are wrong):
                                 //   kProbe* bits below
};
// Probe bits: what the K-loop costs without parts of itself.
constexpr int kProbeResident = 1;     // operands stay in shared memory: loads only for the first STAGES stages of a launch
constexpr int kProbeNoWeights = 2;    // never load weights / metadata
constexpr int kProbeNoActs = 4;       // never load activations
constexpr int kProbeNoMetaCopy = 8;   // no metadata copies into tensor memory
constexpr int kProbeMma2 = 16;        // issue every stage's MMAs twice
constexpr int kProbeMma4 = 32;        // ... four times

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: false if the barrier did not flip within the limit or the CTA is aborting.  The clock
// is only read every 1024 failed polls (the first such reading starts the limit), so a wait that is
// over after a few polls -- every wait of a healthy run -- costs nothing but the polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0ull;
    unsigned int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0ull) {
                t0 = now;
            } else if (now - t0 > *reinterpret_cast<volatile unsigned long long*>(&g_wait_limit_ns)) {
                *abort_flag = 1;
                atomicExch(&g_device_status, static_cast<int>(SBN_ERR_TIMEOUT));
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// Tile store smem -> global (rows beyond the tensor's extent are clipped by the hardware).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int c0, int c1, uint32_t src) {
    asm volatile(
        "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_cp_128x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void mma_i8_dense(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                             uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_i8_sparse(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                              uint32_t e_tmem, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::i8 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (K-major operand): start address, leading/stride byte offsets
// in 16 B units, descriptor version 1, swizzle mode in the top three bits.
constexpr uint64_t kSwzNone = 0, kSwz128 = 2, kSwz64 = 4;
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes,
                                                   uint32_t sbo_bytes, uint64_t swizzle) {
    return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) |
           (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
           (static_cast<uint64_t>(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (swizzle << 61);
}

// Instruction descriptor for kind::i8: D = s32, A = B = signed 8 bit, both K-major.
__host__ __device__ constexpr uint32_t make_idesc_i8(int mma_m, int mma_n, bool sparse) {
    return (sparse ? (1u << 2) : 0u) | (2u << 4) | (1u << 7) | (1u << 10) |
           (static_cast<uint32_t>(mma_n >> 3) << 17) | (static_cast<uint32_t>(mma_m >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------
// Compile-time configuration
// ---------------------------------------------------------------------------------------------
template <bool SPARSE, int BN>
struct GemmConfig {
    static constexpr int A_BYTES = SPARSE ? kBM * (kBK / 2) : kBM * kBK;
    static constexpr int B_BYTES = BN * kBK;
    static constexpr int E_BYTES = SPARSE ? kBM * (kBK / 8) : 0;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
    static constexpr int STAGES_RAW = (kSmemBudget - 1024 - kEpiBytes - kScaleBytes - kBarrierBytes) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr int META_COLS = SPARSE ? 4 * STAGES : 0;
    static constexpr int ACC_STAGES = (2 * BN + META_COLS <= static_cast<int>(kTmemCols)) ? 2 : 1;
    static constexpr int META_COL0 = ACC_STAGES * BN;
    static constexpr uint32_t TX_BYTES = STAGE_BYTES;
    // dynamic smem: 1 KB alignment slack + stages + barriers
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + kEpiBytes + kScaleBytes + kBarrierBytes;
    static_assert(STAGES >= 2, "tile too large for shared memory");
    static_assert(ACC_STAGES * BN + META_COLS <= static_cast<int>(kTmemCols), "TMEM overflow");
};

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <bool SPARSE, int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
bitlinear_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a,
                      const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_e,
                      const __grid_constant__ CUtensorMap tmap_y,
                      const GemmParams p) {
    using Cfg = GemmConfig<SPARSE, BN>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int ACC_STAGES = Cfg::ACC_STAGES;

    pdl_launch_dependents();             // lets the kernels after this one become resident as early as possible
    extern __shared__ uint8_t smem_raw[];
    // 1 KB alignment: required by the 128 B swizzle atoms (8 rows x 128 B)
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_a + STAGES * Cfg::A_BYTES;
    const uint32_t smem_e = smem_b + STAGES * Cfg::B_BYTES;
    const uint32_t smem_epi = smem_base + STAGES * Cfg::STAGE_BYTES;     // 1 KB aligned
    const uint32_t smem_scale = smem_epi + kEpiBytes;                    // float [4][256]
    const uint32_t bar_base = smem_scale + kScaleBytes;                  // 8 B aligned
    const uint32_t bar_full = bar_base;                       // [STAGES]   TMA -> MMA
    const uint32_t bar_empty = bar_full + 8 * STAGES;         // [STAGES]   MMA -> TMA
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;     // [ACC]      MMA -> epilogue
    const uint32_t bar_acc_empty = bar_acc_full + 8 * ACC_STAGES;   // [ACC] epilogue -> MMA
    const uint32_t tmem_slot = bar_acc_empty + 8 * ACC_STAGES;      // 4 B: TMEM base address

    __shared__ int s_abort;
    __shared__ int s_last;
    volatile int* abort_flag = &s_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    const int tiles_m = p.N / kBM;
    const int tiles_t = (p.T + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_t * p.k_splits;
    const int kb_per_split = p.k_blocks_total / p.k_splits;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(bar_acc_full + 8 * a, 1);
            mbar_init(bar_acc_empty + 8 * a, 4);          // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tcgen05_fence_before();
    }
    __syncthreads();
    tcgen05_fence_after();
    // The weights of this CTA's first tile go to L2 while the previous kernel is still finishing: a
    // prefetch into L2 (the point of coherence) cannot make anything stale, whoever wrote them.
    if (threadIdx.x == 32 && blockIdx.x < num_tiles) {
        const int split = blockIdx.x % p.k_splits;
        const int mt0 = (blockIdx.x / p.k_splits) % tiles_m;
        const size_t wt0 = static_cast<size_t>(mt0) * p.k_blocks_total + static_cast<size_t>(split) * kb_per_split;
        prefetch_l2_bulk(static_cast<const char*>(p.w_vals) + wt0 * p.w_tile_bytes, static_cast<uint32_t>(kb_per_split * p.w_tile_bytes));
        if (p.w_meta) prefetch_l2_bulk(static_cast<const char*>(p.w_meta) + wt0 * 2048, static_cast<uint32_t>(kb_per_split * 2048));
    }
    pdl_wait();                          // nothing above reads or writes global memory
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && !p.test_skip_loads) {
            tma_prefetch_desc(&tmap_a);
            tma_prefetch_desc(&tmap_b);
            if constexpr (SPARSE) tma_prefetch_desc(&tmap_e);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int split = tile % p.k_splits;
                const int mt = (tile / p.k_splits) % tiles_m;
                const int tt = (tile / p.k_splits) / tiles_m;
                const int t0 = tt * BN;
                const int kb0 = split * kb_per_split;
                for (int kb = kb0; kb < kb0 + kb_per_split; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = bar_full + 8 * stage;
                    mbar_expect_tx(full, Cfg::TX_BYTES);
                    // operand tiles are stored as smem images (layouts.cuh): 1 KB rows, a few per tile
                    const int wt = mt * p.k_blocks_total + kb;            // weight tile index
                    if constexpr (SPARSE) {
                        tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 8, full);
                        tma_load_2d(smem_e + stage * Cfg::E_BYTES, &tmap_e, 0, wt * 2, full);
                    } else {
                        tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 16, full);
                    }
                    tma_load_2d(smem_b + stage * Cfg::B_BYTES, &tmap_b, 0, kb * p.tb8 + (t0 >> 3), full);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_i8(kBM, BN, SPARSE);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
                for (int kb = 0; kb < kb_per_split; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t a_addr = smem_a + stage * Cfg::A_BYTES;
                    const uint32_t b_addr = smem_b + stage * Cfg::B_BYTES;
                    if constexpr (SPARSE) {
                        const uint32_t e_tmem = tmem_base + static_cast<uint32_t>(Cfg::META_COL0 + 4 * stage);
                        const uint64_t e_desc = make_smem_desc(smem_e + stage * Cfg::E_BYTES, 128, 128, kSwzNone);
                        tcgen05_cp_128x128b(e_tmem, e_desc);
                        const uint64_t a_desc = make_smem_desc(a_addr, 16, 512, kSwz64);
                        const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
#pragma unroll
                        for (int j = 0; j < kBK / 64; ++j) {
                            // per instruction: 32 B of compressed A, 64 B of B, 2 metadata columns
                            mma_i8_sparse(d_tmem, a_desc + static_cast<uint64_t>(2 * j),
                                          b_desc + static_cast<uint64_t>(4 * j), e_tmem + 2 * j, idesc,
                                          (kb | j) != 0 ? 1u : 0u);
                        }
                    } else {
                        const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024, kSwz128);
                        const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
#pragma unroll
                        for (int j = 0; j < kBK / 32; ++j) {
                            mma_i8_dense(d_tmem, a_desc + static_cast<uint64_t>(2 * j),
                                         b_desc + static_cast<uint64_t>(2 * j), idesc,
                                         (kb | j) != 0 ? 1u : 0u);
                        }
                    }
                    tcgen05_commit(bar_empty + 8 * stage);        // smem stage free once read
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tcgen05_commit(bar_acc_full + 8 * acc);           // accumulator complete
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (4 warps)
        // Each warp owns one TMEM lane quarter (32 output features) and works on its own:
        // private scale staging, private double-buffered 32x32 output slab, private TMA stores.
        const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
        const int ew = warp - 2;                          // 0..3: index of this epilogue warp
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const float w_scale = __ldg(p.w_scale);
        uint8_t* const smem_generic = smem_raw + (smem_base - smem_u32(smem_raw));
        const uint32_t slab_u32 = smem_epi + static_cast<uint32_t>(ew * 2 * kEpiWarpBufBytes);
        uint8_t* const slab_ptr = smem_generic + (slab_u32 - smem_base);
        float* const scale_s = reinterpret_cast<float*>(smem_generic + (smem_scale - smem_base)) + ew * 256;
        int acc = 0;
        uint32_t acc_phase = 0;
        int buf = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            const int mt = (tile / p.k_splits) % tiles_m;
            const int tt = (tile / p.k_splits) / tiles_m;
            const int n0 = mt * kBM + quarter * 32;
            const int n = n0 + lane;                              // output feature of this thread
            const int t0 = tt * BN;
            // s absorbs both scales (Eq. 4): stage w_scale * a_scale[t] for the tile's tokens
            __syncwarp();
#pragma unroll
            for (int i = lane; i < BN; i += 32) {
                const int t = t0 + i;
                scale_s[i] = t < p.T ? __fmul_rn(w_scale, __ldg(p.a_scale + t)) : 0.0f;
            }
            const float bias = p.bias ? __ldg(p.bias + n) : 0.0f;
            __syncwarp();
            if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + lane_base + static_cast<uint32_t>(acc * BN + c * 32), r);
                tmem_ld_wait();
                if (c == BN / 32 - 1) {
                    // all of this warp's reads of the accumulator are done: hand it back
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);
                }
                const int tc = t0 + c * 32;
                if (tc >= p.T) continue;                          // whole chunk beyond the last token
                if (p.k_splits > 1) {
                    // split-K: exact int32 accumulation in the scratch (any order gives the same sum)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int t = tc + j;
                        if (t < p.T) atomicAdd(p.split_acc + static_cast<size_t>(t) * p.N + n, static_cast<int>(r[j]));
                    }
                    continue;
                }
                if (p.acc_out) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int t = tc + j;
                        if (t < p.T) p.acc_out[static_cast<size_t>(t) * p.N + n] = static_cast<int>(r[j]);
                    }
                }
                // the slab written two chunks ago must have been read by its TMA store
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
                uint8_t* const slab = slab_ptr + buf * kEpiWarpBufBytes;
                const float4* sc4 = reinterpret_cast<const float4*>(scale_s + c * 32);
                if (p.out_bf16) {
                    uint16_t* o = reinterpret_cast<uint16_t*>(slab) + lane;
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const float4 sc = sc4[j4];
                        float v0 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 0])), sc.x);
                        float v1 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 1])), sc.y);
                        float v2 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 2])), sc.z);
                        float v3 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 3])), sc.w);
                        if (p.bias) { v0 = __fadd_rn(v0, bias); v1 = __fadd_rn(v1, bias); v2 = __fadd_rn(v2, bias); v3 = __fadd_rn(v3, bias); }
                        o[(4 * j4 + 0) * 32] = static_cast<uint16_t>(f32_to_bf16_rne(v0));
                        o[(4 * j4 + 1) * 32] = static_cast<uint16_t>(f32_to_bf16_rne(v1));
                        o[(4 * j4 + 2) * 32] = static_cast<uint16_t>(f32_to_bf16_rne(v2));
                        o[(4 * j4 + 3) * 32] = static_cast<uint16_t>(f32_to_bf16_rne(v3));
                    }
                } else {
                    float* o = reinterpret_cast<float*>(slab) + lane;
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const float4 sc = sc4[j4];
                        float v0 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 0])), sc.x);
                        float v1 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 1])), sc.y);
                        float v2 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 2])), sc.z);
                        float v3 = __fmul_rn(static_cast<float>(static_cast<int>(r[4 * j4 + 3])), sc.w);
                        if (p.bias) { v0 = __fadd_rn(v0, bias); v1 = __fadd_rn(v1, bias); v2 = __fadd_rn(v2, bias); v3 = __fadd_rn(v3, bias); }
                        o[(4 * j4 + 0) * 32] = v0;
                        o[(4 * j4 + 1) * 32] = v1;
                        o[(4 * j4 + 2) * 32] = v2;
                        o[(4 * j4 + 3) * 32] = v3;
                    }
                }
                // generic-proxy writes -> visible to the async proxy, then one lane issues the store
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, n0, tc, slab_u32 + static_cast<uint32_t>(buf * kEpiWarpBufBytes));
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                buf ^= 1;
            }
            if (p.k_splits > 1) {
                // The CTA that adds the last K-slice of an output tile finishes it: dequantise the
                // totals, write y, and leave the scratch zeroed for the next call.
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");              // the four epilogue warps
                const int out_tile = mt + tt * tiles_m;
                if (ew == 0 && lane == 0)
                    s_last = (atomicAdd(p.split_counters + out_tile, 1u) == static_cast<unsigned>(p.k_splits - 1)) ? 1 : 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (s_last) {
                    __threadfence();
                    const int t_end = min(p.T, t0 + BN);
                    for (int tb = t0; tb < t_end; tb += 8) {
                        int a[8];
                        float sc[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {                  // eight independent loads in flight
                            const int t = min(tb + j, t_end - 1);
                            a[j] = __ldcg(p.split_acc + static_cast<size_t>(t) * p.N + n);
                            sc[j] = __fmul_rn(w_scale, __ldg(p.a_scale + t));
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int t = tb + j;
                            if (t < t_end) {
                                const size_t o = static_cast<size_t>(t) * p.N + n;
                                p.split_acc[o] = 0;
                                if (p.acc_out) p.acc_out[o] = a[j];
                                float v = __fmul_rn(static_cast<float>(a[j]), sc[j]);
                                if (p.bias) v = __fadd_rn(v, bias);
                                if (p.out_bf16) static_cast<uint16_t*>(p.y)[o] = static_cast<uint16_t>(f32_to_bf16_rne(v));
                                else static_cast<float*>(p.y)[o] = v;
                            }
                        }
                    }
                    if (ew == 0 && lane == 0) p.split_counters[out_tile] = 0u;
                }
            }
            if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
        // the slabs must stay valid until the stores have read them, and the writes must be done
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
    }

    // teardown: everyone meets here (also on the abort path), then the allocating warp frees TMEM
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace sbn
