// Eq. 4 on CTA pairs: the large-T kernel.
//
// Measured facts that shape it (B200, this kernel family, one CTA pair alone on the GPU):
//   * the time a pipeline stage costs in the TMA unit is  ~64 ns x (number of TMA instructions)
//     + ~2.8 ns per KB, whatever the box shape -- so a stage must be fetched with as few
//     instructions as possible;
//   * an SM sustains roughly 100-120 GB/s of operand ingest, so the tile must reuse operands.
// Hence: two CTAs of a cluster issue one `cta_group::2` MMA (M = 256: each CTA supplies 128
// weight rows and HALF of the activation tile, and keeps its 128 x BN accumulator slice in its
// own TMEM); every CTA runs TWO such M-tiles against the same activation stage; operands are
// stored in HBM as shared-memory images (layouts.cuh) and one 3-D tensor-map box fetches, per
// stage, both of a CTA's weight tiles (and likewise both metadata tiles, and the activation
// atoms) for KBS consecutive 128-column blocks: three instructions per stage (sparse).
//
//   pair tile      512 output features x BN tokens (BN runtime, multiple of 16, <= 240 sparse /
//                  256 dense).  CTA r of the pair owns the weight row blocks 4*mt + 2r + i
//                  (i = 0, 1 = the M-tile); a row block beyond N is skipped.
//   per CTA smem   per stage: A[2 row blocks][KBS] (8 KB sparse | 16 KB dense each),
//                  E[2][KBS] (2 KB each, sparse), B[KBS] (BN/2 rows x 128 B); KBS = 2 (sparse), 1
//   TMEM           M-tile i accumulates in columns [256 i, 256 i + BN); metadata slots (8 columns
//                  each, 2 or 4 of them) at the top of the same 256-column half.  Accumulators are single-buffered: the MMA of the
//                  next tile waits until the epilogue has drained TMEM into registers.
//   warps          0 TMA producer (both CTAs), 1 MMA issuer (leader CTA only; both allocate
//                  TMEM), 2..17 epilogue: warp 2 + e drains M-tile (e >> 2) & 1, TMEM lane
//                  quarter (2 + e) & 3, the even (e < 8) or odd 32-column chunks
//   barriers       full[s]      leader's copy: 1 arrival (leader's expect_tx of BOTH CTAs' bytes),
//                               both CTAs' TMA loads complete_tx on it
//                  empty[s]     every CTA's own copy, arrived by tcgen05.commit multicast
//                  acc_full     every CTA's own copy, commit multicast
//                  acc_empty    leader's copy: 32 arrivals (16 epilogue warps x 2 CTAs)
//
// The same kernel with ONE M-tile per CTA (template parameter MT = 1): the pair tile is 256 features
// wide (CTA r owns row block 2*mt + r), the two 256-column halves of tensor memory alternate as
// accumulators of consecutive tiles (acc_full / acc_empty exist once per half), and all 16 epilogue
// warps drain the one M-tile (four per TMEM lane quarter, chunks c and c + 4) -- so the drain of a
// tile runs under the MMAs of the next one.  It gives up half of the activation reuse; the
// dispatcher uses it for short K and for the dense kernel (see PairConfig).
//
// No TMA multicast is used: every CTA fetches its own boxes.  All waits are bounded.
#pragma once

#include <type_traits>

#include "gemm_tcgen05.cuh"

namespace sbn {

constexpr int kPairEpiWarps = 16;
constexpr int kPairThreads = 32 * (2 + kPairEpiWarps);           // 576 threads, at most 96 registers each
constexpr int kPairEpiBytes = 2 * 256 * 4;                        // per-token scales of the current and the next tile
constexpr int kPairMaxBnSparse = 240;
constexpr int kPairMaxBnDense = 256;

// MT = M-tiles (128-row weight blocks) per CTA.  2: the pair tile is 512 features wide, both M-tiles
// run against the same activation stage (least shared-memory traffic per MMA), accumulators
// single-buffered.  1: 256 features per pair tile, the second half of tensor memory is a second
// accumulator, so the drain of a tile hides under the next tile's MMAs and the tiles are half as
// large -- for short K (few stages per tile) and for tile counts that quantise badly into waves.
template <bool SPARSE, int MT = 2>
struct PairConfig {
    static constexpr int KBS = SPARSE ? 2 : 1;                               // 128-column blocks per stage
    static constexpr int A_TILE = SPARSE ? kBM * (kBK / 2) : kBM * kBK;     // one row block x one k-block
    static constexpr int E_TILE = SPARSE ? kBM * (kBK / 8) : 0;
    static constexpr int B_ROWS_MAX = SPARSE ? kPairMaxBnSparse / 2 : kPairMaxBnDense / 2;
    static constexpr int B_TILE = B_ROWS_MAX * kBK;                          // one k-block of activations
    static constexpr int A_BYTES = MT * KBS * A_TILE;
    static constexpr int E_BYTES = MT * KBS * E_TILE;
    static constexpr int B_BYTES = KBS * B_TILE;
    static constexpr int STAGE_BYTES = A_BYTES + E_BYTES + B_BYTES;
    // the kernel has no static shared memory, so the dynamic part starts 1 KB-aligned (checked)
    static constexpr int STAGES = (232448 - kPairEpiBytes - kBarrierBytes) / STAGE_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + kPairEpiBytes + kBarrierBytes;
    static_assert(STAGE_BYTES % 1024 == 0, "stage must keep 1 KB alignment");
    static_assert(STAGES >= 3, "not enough stages");
    static_assert(!SPARSE || KBS == 2, "the 128x256b metadata copy covers exactly two k-blocks");
    static_assert(SMEM_BYTES <= 232448, "shared memory overflow");
    static_assert(MT == 1 || MT == 2, "M-tiles per CTA");
};

struct PairParams {
    GemmParams g;
    int bn;                       // tokens per tile
};

// int32 accumulator -> fp32, exactly.  The conversion instruction runs at a quarter of the ALU
// rate and the epilogue needs one per output element, so while |acc| < 2^22 (always true for
// K < 32768: |acc| <= 128 K) the integer is added into the mantissa of 1.5 * 2^23 and the
// constant is subtracted again -- full-rate instructions, no rounding anywhere.  Two elements at
// a time: the subtraction and the multiplication by s (Eq. 4) use the packed fp32x2 forms.
template <bool SMALL>
__device__ __forceinline__ void acc2_scaled(uint32_t a0, uint32_t a1, float s0, float s1, float& v0, float& v1) {
    if constexpr (SMALL) {
        uint64_t m, c, sc, d;
        asm("mov.b64 %0, {%1, %2};" : "=l"(m) : "r"(0x4B400000u + a0), "r"(0x4B400000u + a1));
        asm("mov.b64 %0, {%1, %1};" : "=l"(c) : "r"(0xCB400000u));                 // -12582912.0f twice
        asm("mov.b64 %0, {%1, %2};" : "=l"(sc) : "f"(s0), "f"(s1));
        asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(m), "l"(c));
        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(d), "l"(sc));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(v0), "=f"(v1) : "l"(d));
    } else {
        v0 = __fmul_rn(static_cast<float>(static_cast<int>(a0)), s0);
        v1 = __fmul_rn(static_cast<float>(static_cast<int>(a1)), s1);
    }
}

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
// TMA 3-D box load whose completion is counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                                 uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar_cluster_addr)
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
// 128 lanes x 32 B: two 16 B-wide source blocks (LBO apart) land in 8 consecutive TMEM columns.
__device__ __forceinline__ void tcgen05_cp_128x256b_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
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

// Epilogue of one pair tile for one warp, bf16 outputs (see the kernel for the scheme): phase A
// drains this warp's chunks chunk0 + 2 k of the accumulator into packed registers and hands the
// accumulator back, phase B stores them.
template <bool SMALL, int STRIDE>
__device__ __forceinline__ void pair_epilogue_tile_bf16(const GemmParams& p, const int t0, const int n, const float bias,
                                                        const int live, const int full32, const uint32_t t_addr,
                                                        const float* sc_tile, const int lane, const int chunk0,
                                                        const uint32_t acc_empty_leader) {
    constexpr int NK = 8 / STRIDE;                               // chunks per warp: chunk0, chunk0 + STRIDE, ...
    uint32_t packed[NK][16];
    const bool has_bias = p.bias != nullptr;
    // ---- phase A
#pragma unroll
    for (int k = 0; k < NK; ++k) {
        const int i = chunk0 + STRIDE * k;
        if (i < live) {
            const bool half_chunk = (i == full32);                 // the 16-wide tail
            // 16 columns at a time: the tile's packed outputs take most of the registers
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h == 0 || !half_chunk) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(t_addr + static_cast<uint32_t>(i * 32 + h * 16), r);
                    const float2* sc2 = reinterpret_cast<const float2*>(sc_tile + i * 32 + h * 16);   // uniform reads
                    tmem_ld_wait();
                    if (i + STRIDE >= live && (h == 1 || half_chunk)) {
                        // last TMEM read of this warp is complete: hand the accumulator back
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
                    }
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        float v0, v1;
                        const float2 sq = sc2[j >> 1];
                        acc2_scaled<SMALL>(r[j], r[j + 1], sq.x, sq.y, v0, v1);
                        if (has_bias) { v0 = __fadd_rn(v0, bias); v1 = __fadd_rn(v1, bias); }
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(packed[k][(h * 16 + j) >> 1]) : "f"(v1), "f"(v0));
                    }
                }
            }
        }
    }
    // ---- phase B
#pragma unroll
    for (int k = 0; k < NK; ++k) {
        const int i = chunk0 + STRIDE * k;
        if (i < live) {
            const int tc = t0 + i * 32;
            const int cnt = min(p.T - tc, (i == full32) ? 16 : 32);   // live tokens of the chunk (warp-uniform)
            uint16_t* y = static_cast<uint16_t*>(p.y) + static_cast<size_t>(tc) * p.N + n;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const uint32_t pk = packed[k][j >> 1];
                if (j < cnt) __stcs(y, static_cast<uint16_t>(pk & 0xFFFFu));
                if (j + 1 < cnt) __stcs(y + p.N, static_cast<uint16_t>(pk >> 16));
                y += 2 * static_cast<size_t>(p.N);             // running pointer: no table of 32 row addresses
            }
        }
    }
}

// The same for fp32 outputs and / or the raw accumulator dump: these do not fit in registers and
// are stored while the accumulator drains.
template <bool SMALL, int STRIDE>
__device__ __forceinline__ void pair_epilogue_tile_direct(const GemmParams& p, const int t0, const int n, const float bias,
                                                          const int live, const int full32, const uint32_t t_addr,
                                                          const float* sc_tile, const int lane, const int chunk0,
                                                          const uint32_t acc_empty_leader) {
#pragma unroll 1
    for (int i = chunk0; i < live; i += STRIDE) {
        const bool half_chunk = (i == full32);
        const int tc = t0 + i * 32;
        const int cnt = min(p.T - tc, half_chunk ? 16 : 32);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (h == 0 || !half_chunk) {
                uint32_t r[16];
                tmem_ld_32x32b_x16(t_addr + static_cast<uint32_t>(i * 32 + h * 16), r);
                const float2* sc2 = reinterpret_cast<const float2*>(sc_tile + i * 32 + h * 16);
                tmem_ld_wait();
                if (i + STRIDE >= live && (h == 1 || half_chunk)) {
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
                }
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const int jj = h * 16 + j;                    // token inside the chunk
                    const size_t off = static_cast<size_t>(tc + jj) * p.N + n;
                    if (p.acc_out) {
                        if (jj < cnt) p.acc_out[off] = static_cast<int>(r[j]);
                        if (jj + 1 < cnt) p.acc_out[off + p.N] = static_cast<int>(r[j + 1]);
                    }
                    float v0, v1;
                    const float2 sq = sc2[j >> 1];
                    acc2_scaled<SMALL>(r[j], r[j + 1], sq.x, sq.y, v0, v1);
                    if (p.bias) { v0 = __fadd_rn(v0, bias); v1 = __fadd_rn(v1, bias); }
                    if (p.out_bf16) {
                        uint32_t pk;
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(v1), "f"(v0));
                        uint16_t* y = static_cast<uint16_t*>(p.y) + off;
                        if (jj < cnt) y[0] = static_cast<uint16_t>(pk & 0xFFFFu);
                        if (jj + 1 < cnt) y[p.N] = static_cast<uint16_t>(pk >> 16);
                    } else {
                        float* y = static_cast<float*>(p.y) + off;
                        if (jj < cnt) y[0] = v0;
                        if (jj + 1 < cnt) y[p.N] = v1;
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Tensor maps (all over arrays of 1 KB rows of 128 x uint64, see layouts.cuh):
//   tmap_a  [N/128][KB * rows_per_tile][1 KB]   box {1 KB, rows_per_tile * KBS, 2}
//   tmap_e  [N/128][KB * 2][1 KB]               box {1 KB, 2 * KBS, 2}          (sparse)
//   tmap_b  [KB][TB8][1 KB]                     box {1 KB, BN/16, KBS}
template <bool SPARSE, int MT = 2>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
bitlinear_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a,
                           const __grid_constant__ CUtensorMap tmap_b,
                           const __grid_constant__ CUtensorMap tmap_e,
                           const PairParams pp) {
    using Cfg = PairConfig<SPARSE, MT>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int KBS = Cfg::KBS;
    constexpr int A_ROWS = Cfg::A_TILE / 1024;            // 1 KB rows per weight tile
    constexpr int ROWS_PER_TILE = 2 * MT;                  // 128-row weight blocks of a pair tile
    const GemmParams& p = pp.g;
    const int BN = pp.bn;
    const int half_bn = BN >> 1;

    pdl_launch_dependents();             // lets the kernels after this one become resident as early as possible
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = smem_u32(smem_raw);
    if (smem_base & 1023u) {          // swizzled tiles need 1 KB alignment; identical in every CTA
        if (threadIdx.x == 0) atomicExch(&g_device_status, static_cast<int>(SBN_ERR_CUDA));
        return;
    }
    // per stage: A [row block i][k-block j] | E [i][j] | B [j]
    const uint32_t smem_stage0 = smem_base;
    const uint32_t smem_epi = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = smem_epi + kPairEpiBytes;
    const uint32_t bar_full = bar_base;
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;     // [2]: one per accumulator buffer (MT = 2 uses [0])
    const uint32_t bar_acc_empty = bar_acc_full + 16;
    const uint32_t tmem_slot = bar_acc_empty + 16;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (tmem_slot + 8 - smem_base));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();              // 0 = leader of the pair
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    const int n_blocks = p.N >> 7;
    const int tiles_m = (p.N + 128 * ROWS_PER_TILE - 1) / (128 * ROWS_PER_TILE);
    const int tiles_t = (p.T + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_t;
    const int k_blocks = p.k_blocks_total;
    const int k_stages = (k_blocks + KBS - 1) / KBS;      // pipeline stages per tile

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, 2 * kPairEpiWarps);
        }
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
    pdl_wait();                          // nothing above touches global memory
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && !p.test_skip_loads) {
            tma_prefetch_desc(&tmap_a);
            tma_prefetch_desc(&tmap_b);
            if constexpr (SPARSE) tma_prefetch_desc(&tmap_e);
            const uint32_t bytes_per_cta = static_cast<uint32_t>(Cfg::A_BYTES + Cfg::E_BYTES + KBS * half_bn * kBK);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int mt = tile % tiles_m;
                const int tt = tile / tiles_m;
                const int nb0 = mt * ROWS_PER_TILE + static_cast<int>(rank) * MT;   // this CTA's row blocks
                const int t_atom = (tt * BN + static_cast<int>(rank) * half_bn) >> 3;   // this CTA's token half
                for (int ks = 0; ks < k_stages; ++ks) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full_leader = map_to_cta(bar_full + 8 * stage, 0);
                    if (p.probe) {                      // timing experiments (sbn_set_gemm_probe): leave loads out
                        if ((p.probe & kProbeResident) && (tile != pair_id || ks >= STAGES)) {
                            if (rank == 0) mbar_arrive(bar_full + 8 * stage);
                            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                            continue;
                        }
                        const uint32_t skip = ((p.probe & kProbeNoWeights) ? static_cast<uint32_t>(Cfg::A_BYTES + Cfg::E_BYTES) : 0u) +
                                              ((p.probe & kProbeNoActs) ? static_cast<uint32_t>(KBS * half_bn * kBK) : 0u);
                        if (rank == 0) {
                            if (bytes_per_cta > skip) mbar_expect_tx(bar_full + 8 * stage, 2 * (bytes_per_cta - skip));
                            else mbar_arrive(bar_full + 8 * stage);
                        }
                        const uint32_t st_p = smem_stage0 + stage * Cfg::STAGE_BYTES;
                        const int kb_p = ks * KBS;
                        if (!(p.probe & kProbeNoWeights)) {
                            tma_load_3d_pair(st_p, &tmap_a, 0, kb_p * A_ROWS, nb0, full_leader);
                            if constexpr (SPARSE) tma_load_3d_pair(st_p + Cfg::A_BYTES, &tmap_e, 0, kb_p * 2, nb0, full_leader);
                        }
                        if (!(p.probe & kProbeNoActs)) tma_load_3d_pair(st_p + Cfg::A_BYTES + Cfg::E_BYTES, &tmap_b, 0, t_atom, kb_p, full_leader);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * bytes_per_cta);
                    const uint32_t st = smem_stage0 + stage * Cfg::STAGE_BYTES;
                    const int kb = ks * KBS;
                    // boxes that reach beyond the arrays (odd K/128, N % 512 != 0, last tokens) are
                    // zero-filled by the hardware and still count their full size
                    tma_load_3d_pair(st, &tmap_a, 0, kb * A_ROWS, nb0, full_leader);
                    if constexpr (SPARSE) tma_load_3d_pair(st + Cfg::A_BYTES, &tmap_e, 0, kb * 2, nb0, full_leader);
                    tma_load_3d_pair(st + Cfg::A_BYTES + Cfg::E_BYTES, &tmap_b, 0, t_atom, kb, full_leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader)
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = make_idesc_i8(256, BN, SPARSE);
            const uint32_t b_kb_bytes = static_cast<uint32_t>(half_bn * kBK);    // B bytes of one k-block
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;                                      // tiles done by this pair
            uint32_t e_slot = 0;
            const uint32_t e_slots = BN <= 224 ? 4u : 2u;              // 8-column metadata slots above the accumulator
            bool ok = true;
            for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
                const int mt = tile % tiles_m;
                // M-tile i is live if at least the leader's row block exists
                const int mt_count = (MT == 2 && mt * 4 + 1 < n_blocks) ? 2 : 1;
                // MT = 2: one accumulator per M-tile, single-buffered.  MT = 1: the two halves of tensor
                // memory alternate between consecutive tiles.  Either way: wait until the epilogues of
                // both CTAs have drained the accumulator this tile writes.
                const uint32_t buf = (MT == 1) ? (acc_iter & 1u) : 0u;
                const uint32_t acc_phase = (MT == 1) ? ((acc_iter >> 1) & 1u) : (acc_iter & 1u);
                if (!mbar_wait(bar_acc_empty + 8 * buf, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                for (int ks = 0; ks < k_stages; ++ks) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t st = smem_stage0 + stage * Cfg::STAGE_BYTES;
                    const int kb_live = min(KBS, k_blocks - ks * KBS);
                    {
                        uint32_t e_tmem[2] = {0u, 0u};
                        if constexpr (SPARSE) {
                            // every tcgen05 instruction occupies the tensor pipe for ~128 clocks, copies
                            // included: one 128x256b copy brings the metadata of BOTH k-blocks of the
                            // stage (two 2 KB tiles, 2 KB apart) for an M-tile
                            for (int i = 0; i < mt_count; ++i) {
                                e_tmem[i] = tmem_base + static_cast<uint32_t>(i * 256 + 256 - 8 * e_slots + 8 * (e_slot % e_slots));
                                const uint64_t e_desc = make_smem_desc(st + Cfg::A_BYTES + static_cast<uint32_t>(i * KBS * Cfg::E_TILE),
                                                                       Cfg::E_TILE, 128, kSwzNone);
                                if (!(p.probe & kProbeNoMetaCopy)) tcgen05_cp_128x256b_pair(e_tmem[i], e_desc);
                            }
                            ++e_slot;
                        }
                        const int mma_reps = (p.probe & kProbeMma4) ? 4 : ((p.probe & kProbeMma2) ? 2 : 1);     // 1 outside timing experiments
                        for (int rp = 0; rp < mma_reps; ++rp)
                        for (int j = 0; j < kb_live; ++j) {
                            const uint32_t b_addr = st + Cfg::A_BYTES + Cfg::E_BYTES + static_cast<uint32_t>(j) * b_kb_bytes;
                            const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
                            const uint32_t first = (ks | j) == 0 ? 0u : 1u;
                            for (int i = 0; i < mt_count; ++i) {
                                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>((MT == 1 ? buf : i) * 256);
                                const uint32_t a_addr = st + static_cast<uint32_t>((i * KBS + j) * Cfg::A_TILE);
                                if constexpr (SPARSE) {
                                    const uint64_t a_desc = make_smem_desc(a_addr, 16, 512, kSwz64);
#pragma unroll
                                    for (int q = 0; q < kBK / 64; ++q) {
                                        mma_i8_sparse_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * q),
                                                           b_desc + static_cast<uint64_t>(4 * q),
                                                           e_tmem[i] + static_cast<uint32_t>(4 * j + 2 * q), idesc,
                                                           q == 0 ? first : 1u);
                                    }
                                } else {
                                    const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024, kSwz128);
#pragma unroll
                                    for (int q = 0; q < kBK / 32; ++q) {
                                        mma_i8_dense_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * q),
                                                          b_desc + static_cast<uint64_t>(2 * q), idesc,
                                                          q == 0 ? first : 1u);
                                    }
                                }
                            }
                        }
                    }
                    tcgen05_commit_pair(bar_empty + 8 * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tcgen05_commit_pair(bar_acc_full + 8 * buf);
                ++acc_iter;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (16 warps)
        // The accumulators are single-buffered, so the time from "accumulator complete" to
        // "accumulator handed back" is exposed -- and a B200 takes writes at ~3.5 TB/s in total
        // (a plain memset runs at that rate), 24 GB/s per SM: a CTA that stores its 120 KB of
        // bf16 outputs while it drains needs ~5 us, whatever the instruction stream looks like,
        // because all CTAs reach the end of their tiles together.  So the drain does not store:
        //   phase A   TMEM -> registers, scale (Eq. 4), convert, keep the tile's outputs PACKED
        //             IN REGISTERS (bf16: 4 chunks x 32 tokens = 64 registers per thread), hand the
        //             accumulator back -- only arithmetic, ~1.5 us;
        //   phase B   store them while the next tile's MMAs run.
        // Two warps per (M-tile, TMEM lane quarter) take the even / the odd 32-column chunks.
        // A thread owns one output feature (TMEM lane) and 32 tokens of a chunk; y is token-major,
        // so it stores 2 B per token and the warp's 32 lanes make that a contiguous 64 B piece of
        // the token's row -- no transposition, no shared memory.  The per-token scales of the tile
        // are staged in shared memory once per tile and read with uniform 16 B loads.
        // fp32 outputs (and the raw accumulator dump) do not fit in registers: they are stored
        // from phase A directly.
        const int ew = warp - 2;                          // 0..15
        const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
        // MT = 2: M-tile (ew >> 2) & 1, chunks ew >> 3, + 2, + 4, + 6.  MT = 1: chunks ew >> 2, + 4.
        constexpr int STRIDE = (MT == 2) ? 2 : 4;
        const int mtile = (MT == 2) ? ((ew >> 2) & 1) : 0;
        const int chunk0 = (MT == 2) ? (ew >> 3) : (ew >> 2);
        static_assert(kPairEpiWarps == 16, "chunk assignment assumes two warps per lane quarter and M-tile");
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const float w_scale = __ldg(p.w_scale);
        const bool small_acc = k_blocks < 256;            // |acc| <= 128 K < 2^22
        float* const s_scale = reinterpret_cast<float*>(smem_raw + (smem_epi - smem_base));   // [2][256]
        const int et = threadIdx.x - 64;                  // 0..511 among the epilogue threads
        uint32_t tile_par = 0;
        uint32_t acc_iter = 0;
        bool ok = true;
        for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
            const int mt = tile % tiles_m;
            const int tt = tile / tiles_m;
            const int n0 = (mt * ROWS_PER_TILE + static_cast<int>(rank) * MT + mtile) * 128 + quarter * 32;
            const uint32_t buf = (MT == 1) ? (acc_iter & 1u) : 0u;
            const uint32_t acc_phase = (MT == 1) ? ((acc_iter >> 1) & 1u) : (acc_iter & 1u);
            const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty + 8 * buf, 0);
            const int n = n0 + lane;
            const int t0 = tt * BN;
            const bool rows_valid = n0 < p.N;             // warp-uniform (N % 128 == 0)
            const float bias = (p.bias && rows_valid) ? __ldg(p.bias + n) : 0.0f;
            // number of 32-column chunks that hold at least one real token (warp-uniform)
            const int live = rows_valid ? (min(p.T - t0, BN) + 31) >> 5 : 0;
            // a 16-wide last chunk (BN % 32 == 16) is read with a 16-column load: the columns above
            // it hold metadata
            const int full32 = BN >> 5;
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>((MT == 1 ? buf : static_cast<uint32_t>(mtile)) * 256);
            // s of Eq. 4 for the tile's tokens, shared by all epilogue warps (double-buffered over
            // tiles: one named barrier per tile orders the fill against every reader)
            float* const sc_tile = s_scale + tile_par * 256;
            if (et < BN) sc_tile[et] = (t0 + et < p.T) ? __fmul_rn(w_scale, __ldg(p.a_scale + t0 + et)) : 0.0f;
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kPairEpiWarps) : "memory");
            tile_par ^= 1u;
            if (!mbar_wait(bar_acc_full + 8 * buf, acc_phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();

            // bf16 outputs stay in registers until phase B (K >= 32768 takes the plain route: its
            // int32 -> fp32 conversion needs the slow instruction and more registers)
            const bool keep = p.out_bf16 && !p.acc_out && small_acc;
            if (chunk0 >= live) {
                // nothing to read (rows or tokens beyond the matrix): still release the accumulator
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
            } else if (keep) {
                pair_epilogue_tile_bf16<true, STRIDE>(p, t0, n, bias, live, full32, t_addr, sc_tile, lane, chunk0, acc_empty_leader);
            } else {
                if (small_acc) pair_epilogue_tile_direct<true, STRIDE>(p, t0, n, bias, live, full32, t_addr, sc_tile, lane, chunk0, acc_empty_leader);
                else pair_epilogue_tile_direct<false, STRIDE>(p, t0, n, bias, live, full32, t_addr, sc_tile, lane, chunk0, acc_empty_leader);
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
}

}  // namespace sbn
