// Eq. 4 on CTA pairs: the large-T kernel.
//
// Why pairs: an SM can take in about 64 B per clock from L2.  At the sparse int8 rate a CTA that
// owns a 128 x 256 output tile needs ~160 B/clk of operands, so single-CTA tiles are held at a
// third of the tensor peak by operand ingest, not by the MMA.  Here two CTAs of a cluster issue
// one `cta_group::2` MMA (M = 256: each CTA supplies 128 weight rows and HALF of the activation
// tile, and keeps its 128 x BN accumulator slice in its own TMEM), and every CTA runs TWO such
// M-tiles against the same activation stage.  Per CTA and per unit of K that is
// 2*(64+8) + BN/2 bytes (sparse) for 256 x BN MACs: ~68 B/clk at the sparse peak for BN = 240.
//
//   pair tile      512 output features x BN tokens (BN runtime, multiple of 16, <= 240 sparse /
//                  256 dense); the last feature tile may hold only one M-tile
//   per CTA smem   per stage: 2 x A (128 rows x 64 B sparse | 128 B dense), 2 x E (128 x 16 B),
//                  B (BN/2 rows x 128 B); ring of STAGES stages
//   TMEM           M-tile i accumulates in columns [256 i, 256 i + BN); metadata slots in columns
//                  [256 i + 240, 256 i + 256).  Accumulators are single-buffered: the MMA of the
//                  next tile waits until the epilogue has drained TMEM into registers.
//   warps          0 TMA producer (both CTAs), 1 MMA issuer (leader CTA only; both allocate
//                  TMEM), 2..9 epilogue: warps 2-5 drain M-tile 0, warps 6-9 M-tile 1
//   barriers       full[s]      leader's copy: 1 arrival (leader's expect_tx of BOTH CTAs' bytes),
//                               both CTAs' TMA loads complete_tx on it
//                  empty[s]     every CTA's own copy, arrived by tcgen05.commit multicast
//                  acc_full     every CTA's own copy, commit multicast
//                  acc_empty    leader's copy: 16 arrivals (8 epilogue warps x 2 CTAs)
//
// No TMA multicast is used: every CTA fetches its own boxes.  All waits are bounded.
#pragma once

#include "gemm_tcgen05.cuh"

namespace sbn {

constexpr int kPairThreads = 320;
constexpr int kPairEpiWarps = 8;
constexpr int kPairSlabBytes = 16 * 32 * 4;                       // 16 tokens x 32 features fp32
constexpr int kPairEpiBytes = kPairEpiWarps * 2 * kPairSlabBytes; // double buffered per warp
constexpr int kPairMaxBnSparse = 240;
constexpr int kPairMaxBnDense = 256;

template <bool SPARSE>
struct PairConfig {
    static constexpr int A_TILE = SPARSE ? kBM * (kBK / 2) : kBM * kBK;     // one M-tile half
    static constexpr int E_TILE = SPARSE ? kBM * (kBK / 8) : 0;
    static constexpr int B_TILE = 128 * kBK;                                 // up to 128 token rows
    static constexpr int STAGE_BYTES = 2 * A_TILE + 2 * E_TILE + B_TILE;
    static constexpr int STAGES = (232448 - 1024 - kPairEpiBytes - kBarrierBytes) / STAGE_BYTES;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + kPairEpiBytes + kBarrierBytes;
    static_assert(STAGES >= 3, "not enough stages");
    static_assert(SMEM_BYTES <= 232448, "shared memory overflow");
};

struct PairParams {
    GemmParams g;
    int bn;                       // tokens per tile
};

// ---- cluster / pair PTX ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared variable in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load whose completion is counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// Arrive on the barrier at this offset in both CTAs of the pair once all prior MMAs are done.
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tcgen05_cp_128x128b_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void mma_i8_dense_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                                  uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_i8_sparse_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                                   uint32_t e_tmem, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::i8 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

// ---------------------------------------------------------------------------------------------
template <bool SPARSE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
bitlinear_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a,
                           const __grid_constant__ CUtensorMap tmap_b,
                           const __grid_constant__ CUtensorMap tmap_e,
                           const __grid_constant__ CUtensorMap tmap_y,
                           const PairParams pp) {
    using Cfg = PairConfig<SPARSE>;
    constexpr int STAGES = Cfg::STAGES;
    const GemmParams& p = pp.g;
    const int BN = pp.bn;
    const int half_bn = BN >> 1;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // per stage: [A0][A1][E0][E1][B]
    const uint32_t smem_stage0 = smem_base;
    const uint32_t smem_epi = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = smem_epi + kPairEpiBytes;
    const uint32_t bar_full = bar_base;
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;
    const uint32_t bar_acc_empty = bar_acc_full + 8;
    const uint32_t tmem_slot = bar_acc_empty + 8;

    __shared__ int s_abort;
    volatile int* abort_flag = &s_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();              // 0 = leader of the pair
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    const int tiles_m = (p.N + 511) / 512;
    const int tiles_t = (p.T + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_t;
    const int k_blocks = p.k_blocks_total;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 2 * kPairEpiWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kTmemCols);
        tcgen05_fence_before();
    }
    __syncthreads();
    cluster_sync_all();                  // the peer's barriers exist before anything is signalled
    tcgen05_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmap_a);
            tma_prefetch_desc(&tmap_b);
            if constexpr (SPARSE) tma_prefetch_desc(&tmap_e);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int mt = tile % tiles_m;
                const int tt = tile / tiles_m;
                const int m0 = mt * 512;
                const int mt_count = (m0 + 256 < p.N) ? 2 : 1;
                const int t_row = tt * BN + static_cast<int>(rank) * half_bn;    // this CTA's token half
                const uint32_t bytes_per_cta = static_cast<uint32_t>(mt_count * (Cfg::A_TILE + Cfg::E_TILE) + half_bn * kBK);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full_leader = map_to_cta(bar_full + 8 * stage, 0);
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * bytes_per_cta);
                    const uint32_t st = smem_stage0 + stage * Cfg::STAGE_BYTES;
                    for (int i = 0; i < mt_count; ++i) {
                        const int row = m0 + i * 256 + static_cast<int>(rank) * 128;
                        if constexpr (SPARSE) {
                            tma_load_2d_pair(st + i * Cfg::A_TILE, &tmap_a, kb * (kBK / 2), row, full_leader);
                            tma_load_2d_pair(st + 2 * Cfg::A_TILE + i * Cfg::E_TILE, &tmap_e, kb * (kBK / 8), row, full_leader);
                        } else {
                            tma_load_2d_pair(st + i * Cfg::A_TILE, &tmap_a, kb * kBK, row, full_leader);
                        }
                    }
                    tma_load_2d_pair(st + 2 * Cfg::A_TILE + 2 * Cfg::E_TILE, &tmap_b, kb * kBK, t_row, full_leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader)
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = make_idesc_i8(256, BN, SPARSE);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int mt = tile % tiles_m;
                const int m0 = mt * 512;
                const int mt_count = (m0 + 256 < p.N) ? 2 : 1;
                // single-buffered accumulators: wait until the epilogues of both CTAs drained them
                if (!mbar_wait(bar_acc_empty, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t st = smem_stage0 + stage * Cfg::STAGE_BYTES;
                    const uint32_t b_addr = st + 2 * Cfg::A_TILE + 2 * Cfg::E_TILE;
                    const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
                    for (int i = 0; i < mt_count; ++i) {
                        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(i * 256);
                        const uint32_t a_addr = st + i * Cfg::A_TILE;
                        if constexpr (SPARSE) {
                            const uint32_t e_tmem = tmem_base + static_cast<uint32_t>(i * 256 + 240 + 4 * (kb & 3));
                            const uint64_t e_desc = make_smem_desc(st + 2 * Cfg::A_TILE + i * Cfg::E_TILE, 128, 128, kSwzNone);
                            tcgen05_cp_128x128b_pair(e_tmem, e_desc);
                            const uint64_t a_desc = make_smem_desc(a_addr, 16, 512, kSwz64);
#pragma unroll
                            for (int j = 0; j < kBK / 64; ++j) {
                                mma_i8_sparse_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * j),
                                                   b_desc + static_cast<uint64_t>(4 * j), e_tmem + 2 * j, idesc,
                                                   (kb | j) != 0 ? 1u : 0u);
                            }
                        } else {
                            const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024, kSwz128);
#pragma unroll
                            for (int j = 0; j < kBK / 32; ++j) {
                                mma_i8_dense_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * j),
                                                  b_desc + static_cast<uint64_t>(2 * j), idesc,
                                                  (kb | j) != 0 ? 1u : 0u);
                            }
                        }
                    }
                    tcgen05_commit_pair(bar_empty + 8 * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tcgen05_commit_pair(bar_acc_full);
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (8 warps)
        const int ew = warp - 2;                          // 0..7
        const int mtile = ew >> 2;                        // which M-tile this warp drains
        const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const float w_scale = __ldg(p.w_scale);
        const uint32_t slab_u32 = smem_epi + static_cast<uint32_t>(ew * 2 * kPairSlabBytes);
        uint8_t* const slab_ptr = smem_raw + (slab_u32 - smem_u32(smem_raw));
        const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
        uint32_t acc_phase = 0;
        int buf = 0;
        bool ok = true;
        for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
            const int mt = tile % tiles_m;
            const int tt = tile / tiles_m;
            const int m0 = mt * 512;
            const int n0 = m0 + mtile * 256 + static_cast<int>(rank) * 128 + quarter * 32;
            const int n = n0 + lane;
            const int t0 = tt * BN;
            const bool rows_valid = n0 < p.N;             // warp-uniform (N % 128 == 0)
            const float bias = (p.bias && rows_valid) ? __ldg(p.bias + n) : 0.0f;
            if (!mbar_wait(bar_acc_full, acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            const int chunks = BN >> 4;
#pragma unroll 1
            for (int c = 0; c < chunks; ++c) {
                const int tc = t0 + c * 16;
                const bool active = rows_valid && tc < p.T;
                uint32_t r[16];
                float my_scale = 0.0f;
                if (active) {
                    const int t = tc + (lane & 15);
                    if (t < p.T) my_scale = __fmul_rn(w_scale, __ldg(p.a_scale + t));
                    tmem_ld_32x32b_x16(tmem_base + lane_base + static_cast<uint32_t>(mtile * 256 + c * 16), r);
                    tmem_ld_wait();
                }
                if (c == chunks - 1) {
                    // this warp has read everything it needs from the accumulators
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
                }
                if (!active) continue;
                if (p.acc_out) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = tc + j;
                        if (t < p.T) p.acc_out[static_cast<size_t>(t) * p.N + n] = static_cast<int>(r[j]);
                    }
                }
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
                uint8_t* const slab = slab_ptr + buf * kPairSlabBytes;
                if (p.out_bf16) {
                    uint16_t* o = reinterpret_cast<uint16_t*>(slab) + lane;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float sc = __shfl_sync(0xFFFFFFFFu, my_scale, j);
                        float v = __fmul_rn(static_cast<float>(static_cast<int>(r[j])), sc);
                        if (p.bias) v = __fadd_rn(v, bias);
                        o[j * 32] = static_cast<uint16_t>(f32_to_bf16_rne(v));
                    }
                } else {
                    float* o = reinterpret_cast<float*>(slab) + lane;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float sc = __shfl_sync(0xFFFFFFFFu, my_scale, j);
                        float v = __fmul_rn(static_cast<float>(static_cast<int>(r[j])), sc);
                        if (p.bias) v = __fadd_rn(v, bias);
                        o[j * 32] = v;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, n0, tc, slab_u32 + static_cast<uint32_t>(buf * kPairSlabBytes));
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                buf ^= 1;
            }
            acc_phase ^= 1u;
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
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
}

}  // namespace sbn
