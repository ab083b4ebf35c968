// D[M][Nn] = A[M][Kc] * B[Nn][Kc]^T in bf16 with fp32 accumulation on the 5th-generation tensor cores --
// the two contractions of the layer's backward pass (Sec. 2.3, Eq. 5: dX = dY w_masked with K-major
// operands, dW = dY^T x_q with MN-major ones; backward_prep.cuh makes the bf16 operands).
//
// Same skeleton as the int8 CTA-pair kernel (gemm_pair_tcgen05.cuh): two CTAs of a cluster issue one
// `tcgen05.mma.cta_group::2.kind::f16` (M = 256: each CTA supplies 128 rows of A and half of the B tile
// and keeps its 128 x BN slice of the accumulator in its own tensor memory), persistent over output tiles
// of 256 x BN (BN runtime, multiple of 16, <= 256), operands fetched by TMA (plain row-major tensors,
// 128-byte swizzle: a box of 64 bf16 x rows IS the K-major shared-memory image), the full barrier of a
// stage lives in the leader CTA and collects both CTAs' bytes, `tcgen05.commit ... multicast::cluster`
// releases stages and publishes accumulators in both CTAs.  The two 256-column halves of tensor memory
// alternate as accumulators, so the epilogue of a tile (8 warps: TMEM -> registers -> optional scale ->
// row-major fp32 or bf16 stores; a thread owns an output row and writes 128 B or 64 B runs of it) runs
// under the next tile's MMAs.  No TMA multicast.  All waits are bounded.
//
//   warps        0 TMA producer (both CTAs), 1 MMA issuer (leader CTA only; both allocate TMEM),
//                2..9 epilogue: warp w reads TMEM lane quarter w % 4, the even (w < 6) or odd 32-column chunks
//   per stage    A 128 rows x 128 B (16 KB) | B BN/2 rows x 128 B (<= 16 KB): K step of 64 elements,
//                four MMAs of K = 16
#pragma once

#include "gemm_pair_tcgen05.cuh"

namespace sbn {

constexpr int kBf16EpiWarps = 8;
constexpr int kBf16Threads = 32 * (2 + kBf16EpiWarps);
constexpr int kBf16StageA = 128 * 128;                      // bytes
constexpr int kBf16StageB = 128 * 128;                      // bytes reserved (BN/2 <= 128 rows)
constexpr int kBf16StageBytes = kBf16StageA + kBf16StageB;
constexpr int kBf16Stages = 6;
constexpr int kBf16SmemBytes = kBf16Stages * kBf16StageBytes + kBarrierBytes;
static_assert(kBf16SmemBytes <= 232448, "shared memory overflow");

struct Bf16GemmParams {
    int M, Nn, Kc;               // output rows, output columns, contraction length (elements)
    int bn;                      // output columns per tile
    void* out;                   // [M][Nn] row-major, fp32 or bf16
    int out_bf16;
    const float* scale;          // device, one fp32, or null: the result is multiplied by bf16(scale)
    // Two launches of this kernel that do not depend on each other (dW and dX of one backward call) share
    // the machine at the seam: the first one's last wave leaves pairs idle, the second one's CTAs move in as
    // soon as pairs are free instead of waiting for the whole grid.
    //   first launch:  signal_after_wait -- it lets its dependents go only after its own dependency wait, so
    //                  that whatever it waited for is complete for them too;
    //   second launch: wait_at_end -- no dependency wait before its work (its inputs are complete by the rule
    //                  above), but one before it exits: it is not complete before the first launch is, and the
    //                  kernels after it in the stream see both results.
    int signal_after_wait = 0;
    int wait_at_end = 0;
};

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
        : "memory");
}
__device__ __forceinline__ void mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Instruction descriptor for kind::f16: D = fp32, A = B = bf16; both K-major, or both MN-major (the
// contraction index is the SLOW index of the operands in memory: bits 15 / 16).
__host__ __device__ constexpr uint32_t make_idesc_bf16(int mma_m, int mma_n, bool mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (mn_major ? ((1u << 15) | (1u << 16)) : 0u) |
           (static_cast<uint32_t>(mma_n >> 3) << 17) | (static_cast<uint32_t>(mma_m >> 4) << 24);
}

// MN = false (K-major operands):  tmap_a: [M][Kc] bf16, box {64, 128};  tmap_b: [Nn][Kc] bf16, box {64, bn / 2}.
// MN = true (MN-major operands: A is stored [Kc][M], B is stored [Kc][Nn], i.e. D = A^T B without a
// transposed copy of either):  tmap_a: [Kc][M], box {64 of M, 64 of Kc};  tmap_b: [Kc][Nn], box {64, 64};
// bn must be 128 or 256.  A box of 64 contraction rows x 128 B is the MN-major shared-memory image of a
// block of 64 output rows (or columns): 8-row groups 1 KB apart along the contraction (the stride offset),
// blocks 8 KB apart (the leading offset); an MMA of K = 16 starts 2 KB further per step.
template <bool MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kBf16Threads, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Bf16GemmParams p) {
    constexpr int STAGES = kBf16Stages;
    const int BN = p.bn;
    const int half_bn = BN >> 1;

    if (!p.signal_after_wait) pdl_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = smem_u32(smem_raw);
    if (smem_base & 1023u) {          // swizzled tiles need 1 KB alignment; identical in every CTA
        if (threadIdx.x == 0) atomicExch(&g_device_status, static_cast<int>(SBN_ERR_CUDA));
        return;
    }
    const uint32_t bar_base = smem_base + STAGES * kBf16StageBytes;
    const uint32_t bar_full = bar_base;
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;     // [2]
    const uint32_t bar_acc_empty = bar_acc_full + 16;         // [2]
    const uint32_t tmem_slot = bar_acc_empty + 16;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (tmem_slot + 8 - smem_base));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    const int tiles_m = (p.M + 255) / 256;
    const int tiles_n = (p.Nn + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int k_stages = (p.Kc + 63) / 64;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, 2 * kBf16EpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kTmemCols);
        tcgen05_fence_before();
    }
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    if (!p.wait_at_end) pdl_wait();      // nothing above touches global memory
    if (p.signal_after_wait) pdl_launch_dependents();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmap_a);
            tma_prefetch_desc(&tmap_b);
            const uint32_t bytes_per_cta = static_cast<uint32_t>(kBf16StageA + half_bn * 128);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int m0 = (tile % tiles_m) * 256 + static_cast<int>(rank) * 128;
                const int n0 = (tile / tiles_m) * BN + static_cast<int>(rank) * half_bn;
                for (int ks = 0; ks < k_stages; ++ks) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full_leader = map_to_cta(bar_full + 8 * stage, 0);
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * bytes_per_cta);
                    const uint32_t st = smem_base + stage * kBf16StageBytes;
                    // rows or columns beyond the tensors are zero-filled by the hardware and still count their full size
                    if constexpr (MN) {
                        tma_load_2d_pair(st, &tmap_a, m0, ks * 64, full_leader);
                        tma_load_2d_pair(st + 8192, &tmap_a, m0 + 64, ks * 64, full_leader);
                        for (int j = 0; j < half_bn / 64; ++j)
                            tma_load_2d_pair(st + kBf16StageA + j * 8192, &tmap_b, n0 + 64 * j, ks * 64, full_leader);
                    } else {
                        tma_load_2d_pair(st, &tmap_a, ks * 64, m0, full_leader);
                        tma_load_2d_pair(st + kBf16StageA, &tmap_b, ks * 64, n0, full_leader);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader)
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = make_idesc_bf16(256, BN, MN);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const uint32_t buf = acc_iter & 1u;
                const uint32_t acc_phase = (acc_iter >> 1) & 1u;
                if (!mbar_wait(bar_acc_empty + 8 * buf, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256u;
                for (int ks = 0; ks < k_stages; ++ks) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t st = smem_base + stage * kBf16StageBytes;
                    const uint64_t a_desc = MN ? make_smem_desc(st, 8192, 1024, kSwz128) : make_smem_desc(st, 16, 1024, kSwz128);
                    const uint64_t b_desc = MN ? make_smem_desc(st + kBf16StageA, 8192, 1024, kSwz128) : make_smem_desc(st + kBf16StageA, 16, 1024, kSwz128);
                    constexpr uint64_t kStep = MN ? (2048 >> 4) : (32 >> 4);      // K = 16 elements per instruction: 16 rows, or 32 B along a row
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        mma_bf16_pair(d_tmem, a_desc + kStep * q, b_desc + kStep * q, idesc, (ks | q) != 0 ? 1u : 0u);
                    tcgen05_commit_pair(bar_empty + 8 * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tcgen05_commit_pair(bar_acc_full + 8 * buf);
                ++acc_iter;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (8 warps)
        const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
        const int parity = (warp - 2) >> 2;               // even or odd 32-column chunks
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        float scale = 1.0f;
        if (p.scale != nullptr) scale = __uint_as_float(f32_to_bf16_rne(__ldg(p.scale)) << 16);    // the scale as a bf16 run holds it
        uint32_t acc_iter = 0;
        bool ok = true;
        for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
            const int m = (tile % tiles_m) * 256 + static_cast<int>(rank) * 128 + quarter * 32 + lane;
            const int n_tile = (tile / tiles_m) * BN;
            const uint32_t buf = acc_iter & 1u;
            const uint32_t acc_phase = (acc_iter >> 1) & 1u;
            const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty + 8 * buf, 0);
            if (!mbar_wait(bar_acc_full + 8 * buf, acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + buf * 256u;
            const int chunks = (BN + 31) >> 5;            // a last chunk of 16 columns when BN % 32 == 16
            int my_last = -1;
            for (int c = parity; c < chunks; c += 2) my_last = c;
            if (my_last < 0) {
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
            }
#pragma unroll 1
            for (int c = parity; c < chunks; c += 2) {
                const int width = min(32, BN - c * 32);   // 32 or 16
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h * 16 < width) {
                        uint32_t r[16];
                        tmem_ld_32x32b_x16(t_addr + static_cast<uint32_t>(c * 32 + h * 16), r);
                        tmem_ld_wait();
                        if (c == my_last && (h == 1 || width == 16)) {
                            tcgen05_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
                        }
                        const int n = n_tile + c * 32 + h * 16;
                        if (m < p.M && n < p.Nn) {        // Nn % 16 == 0: a run of 16 columns is in or out as a whole
                            if (p.out_bf16) {
                                uint32_t pk[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    const float v0 = __fmul_rn(__uint_as_float(r[2 * j]), scale), v1 = __fmul_rn(__uint_as_float(r[2 * j + 1]), scale);
                                    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[j]) : "f"(v1), "f"(v0));
                                }
                                uint4* o = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + static_cast<size_t>(m) * p.Nn + n);
                                o[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                o[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                            } else {
                                float4* o = reinterpret_cast<float4*>(static_cast<float*>(p.out) + static_cast<size_t>(m) * p.Nn + n);
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    o[j] = make_float4(__fmul_rn(__uint_as_float(r[4 * j]), scale), __fmul_rn(__uint_as_float(r[4 * j + 1]), scale),
                                                       __fmul_rn(__uint_as_float(r[4 * j + 2]), scale), __fmul_rn(__uint_as_float(r[4 * j + 3]), scale));
                            }
                        }
                    }
                }
            }
            ++acc_iter;
        }
    }

    // teardown: nobody leaves while the peer may still touch this CTA's smem, barriers or TMEM
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
    if (p.wait_at_end) pdl_wait();
}

}  // namespace sbn
