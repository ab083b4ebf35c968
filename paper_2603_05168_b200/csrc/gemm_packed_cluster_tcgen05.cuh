// Eq. 4 for few tokens from PACKED weights (bitpack24.cuh: kept values at two bits each next to
// the unchanged metadata, 2 bits per weight, 4 KB per 128 x 128 block instead of 10 KB).
//
// On matrices of 7B-class size the few-token GEMM is bound by the weight stream (28 MB per call at
// 5 bits per weight).  Here the CTA fetches the 2 KB value tiles and the 2 KB metadata tiles with
// bulk copies (no tensor map: a tile is one contiguous block), and its four epilogue warps -- idle
// during the K-loop otherwise -- expand every value tile into the 64 B-swizzled shared-memory image
// the sparse MMA reads: a thread takes 8 groups (one word in, 16 bytes out) at three ALU
// instructions per group, no table, every shared-memory access conflict-free.  Everything else is
// the cluster split-K kernel of gemm_splitk_cluster_tcgen05.cuh: K slices over the S CTAs of a
// cluster, partial sums reduced through distributed shared memory with st.async, two CTAs per SM.
//
//   warp 0, lane 0   bulk copies of packed tiles (8-deep ring; the first 8 before the dependency
//                    wait, like the weights of the int8-held kernel), TMA loads of the activations
//   warp 1, lane 0   per k-block: wait for the expanded stage and the activations, metadata copy,
//                    two sparse MMAs, commit
//   warps 2..5       expand k-block after k-block (the first STAGES of them before the dependency
//                    wait), then the reduce-scatter and finish as in the int8-held kernel
#pragma once

#include "bitpack24.cuh"
#include "gemm_splitk_cluster_tcgen05.cuh"

namespace sbn {

struct PackedSplitConfig {
    static constexpr int BN = 32;
    static constexpr int A_BYTES = kBM * (kBK / 2);
    static constexpr int B_BYTES = BN * kBK;
    static constexpr int E_BYTES = kBM * (kBK / 8);
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
    static constexpr int STAGES = 4;
    static constexpr int RAW_STAGES = 8;
    static constexpr int RAW_SLOT_BYTES = kVals2TileBytes + 2048;          // value tile | metadata tile
    static constexpr int RAW_BYTES = RAW_STAGES * RAW_SLOT_BYTES;
    static constexpr int REDUCE_BYTES = (BN + 4) * kBM * 4;               // S * ceil(BN / S) token slots, S in {2, 3, 4, 8}
    static constexpr int BAR_BYTES = 512;
    static constexpr int META_COL0 = BN;
    static constexpr uint32_t TMEM_COLS = 64;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + REDUCE_BYTES + RAW_BYTES + BAR_BYTES;
    static_assert(BN + 4 * STAGES <= 64, "tensor memory columns");
    static_assert(SMEM_BYTES <= 232448 / 2 - 1024, "two CTAs per SM");
};

// Plain (untiled) bulk copy global -> shared, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gmem_src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__global__ void __launch_bounds__(kSplitThreads, 2)
bitlinear_gemm_packed_cluster_kernel(const __grid_constant__ CUtensorMap tmap_b, const GemmParams p) {
    using Cfg = PackedSplitConfig;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int RAW = Cfg::RAW_STAGES;
    constexpr int BN = Cfg::BN;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_a + STAGES * Cfg::A_BYTES;
    const uint32_t smem_e = smem_b + STAGES * Cfg::B_BYTES;
    const uint32_t smem_red = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t smem_pk = smem_red + Cfg::REDUCE_BYTES;                 // ring of packed tiles
    const uint32_t bar_base = smem_pk + Cfg::RAW_BYTES;
    const uint32_t bar_full = bar_base;                                    // activations of a stage have landed
    const uint32_t bar_empty = bar_full + 8 * STAGES;                      // the MMAs of a stage are done
    const uint32_t bar_exp = bar_empty + 8 * STAGES;                       // a stage's weights are expanded (128 arrivals)
    const uint32_t bar_pk_full = bar_exp + 8 * STAGES;                     // a packed tile has landed
    const uint32_t bar_pk_empty = bar_pk_full + 8 * RAW;                   // ... and has been read (128 arrivals)
    const uint32_t bar_acc_full = bar_pk_empty + 8 * RAW;
    const uint32_t bar_red = bar_acc_full + 8;
    const uint32_t tmem_slot = bar_red + 8;

    __shared__ int s_abort;
    volatile int* abort_flag = &s_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t S = cluster_nctarank();
    const int tile = blockIdx.x / static_cast<int>(S);
    const int tiles_m = p.N / kBM;
    const int mt = tile % tiles_m;
    const int tt = tile / tiles_m;
    const int t0 = tt * BN;
    const int q = (p.k_blocks_total + static_cast<int>(S) - 1) / static_cast<int>(S);
    const int kb0 = min(p.k_blocks_total, static_cast<int>(rank) * q);
    const int kb1 = min(p.k_blocks_total, kb0 + q);
    const int nblk = kb1 - kb0;
    const int tok_per_cta = (BN + static_cast<int>(S) - 1) / static_cast<int>(S);
    const int tile_tokens = min(BN, p.T - t0);
    const int my_tokens = max(0, (tile_tokens - static_cast<int>(rank) + static_cast<int>(S) - 1) / static_cast<int>(S));
    const size_t tile0 = static_cast<size_t>(mt) * p.k_blocks_total + kb0;
    const uint8_t* v2_tiles = static_cast<const uint8_t*>(p.w_vals) + tile0 * kVals2TileBytes;
    const uint8_t* me_tiles = static_cast<const uint8_t*>(p.w_meta) + tile0 * 2048;
    constexpr uint32_t kSlot = Cfg::RAW_SLOT_BYTES;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
            mbar_init(bar_exp + 8 * s, 128);
        }
        for (int s = 0; s < RAW; ++s) {
            mbar_init(bar_pk_full + 8 * s, 1);
            mbar_init(bar_pk_empty + 8 * s, 128);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_red, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar_red, static_cast<uint32_t>(my_tokens) * S * (kBM * 4));
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tcgen05_fence_before();
    }
    __syncthreads();
    tcgen05_fence_after();
    cluster_arrive();

    // Packed tiles of the first RAW k-blocks: fetched before the dependency wait (weights only; safe
    // for the reason given in sbn_common.cuh).
    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmap_b);
        const int n_pre = min(RAW, nblk);
        for (int i = 0; i < n_pre; ++i) {
            mbar_expect_tx(bar_pk_full + 8 * i, kSlot);
            bulk_load(smem_pk + i * kSlot, v2_tiles + static_cast<size_t>(i) * kVals2TileBytes, kVals2TileBytes, bar_pk_full + 8 * i);
            bulk_load(smem_pk + i * kSlot + kVals2TileBytes, me_tiles + static_cast<size_t>(i) * 2048, 2048, bar_pk_full + 8 * i);
        }
        if (nblk > n_pre) {
            prefetch_l2_bulk(v2_tiles + static_cast<size_t>(n_pre) * kVals2TileBytes, static_cast<uint32_t>((nblk - n_pre) * kVals2TileBytes));
            prefetch_l2_bulk(me_tiles + static_cast<size_t>(n_pre) * 2048, static_cast<uint32_t>((nblk - n_pre) * 2048));
        }
    }

    bool ok = true;
    const uint8_t* pk_generic = smem_raw + (smem_pk - smem_u32(smem_raw));
    // Expands k-block `blk` of this CTA's slice into its stage.  Thread (row, 16 B chunk): one word of
    // packed values in, one chunk of the swizzled value image out, four rows per thread; the metadata
    // tile is copied as it is.  A warp reads 512 contiguous bytes and writes 8 whole 64 B rows.
    auto expand_block = [&](int blk) {
        const int stage = blk % STAGES, slot = blk % RAW;
        const uint32_t tix = threadIdx.x - 64;
        const uint32_t c = tix & 3u;
        if (!mbar_wait(bar_pk_full + 8 * slot, static_cast<uint32_t>(blk / RAW) & 1u, abort_flag)) { ok = false; return; }
        if (blk >= STAGES && !mbar_wait(bar_empty + 8 * stage, static_cast<uint32_t>(blk / STAGES - 1) & 1u, abort_flag)) { ok = false; return; }
        const uint32_t* src = reinterpret_cast<const uint32_t*>(pk_generic + slot * kSlot);
        uint32_t x[4], m[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t r = (tix >> 2) + 32u * i;
            x[i] = src[r * 4 + c];
            m[i] = src[kVals2TileBytes / 4 + r * 4 + c];
        }
        mbar_arrive(bar_pk_empty + 8 * slot);                             // the packed tiles may be overwritten
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t r = (tix >> 2) + 32u * i;
            uint32_t o[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // one byte = t0 t1 t0' t1' at two bits each -> four bytes, then t - 1 per byte
                const uint32_t b = (x[i] >> (8 * k)) & 0xFFu;
                const uint32_t u = b | (b << 6);
                o[k] = __vsub4((u | (u << 12)) & 0x03030303u, 0x01010101u);
            }
            st_shared_v4(smem_a + stage * Cfg::A_BYTES + r * 64u + ((c ^ ((r >> 1) & 3u)) << 4), o[0], o[1], o[2], o[3]);
            asm volatile("st.shared.u32 [%0], %1;" ::"r"(smem_e + stage * Cfg::E_BYTES + r * 16u + 4u * c), "r"(m[i]) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic-proxy writes -> tensor core reads
        mbar_arrive(bar_exp + 8 * stage);
    };
    const int n_exp_pre = min(STAGES, nblk);
    if (warp >= 2) {
        for (int blk = 0; blk < n_exp_pre && ok; ++blk) expand_block(blk);
    }

    pdl_wait();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            for (int blk = 0; blk < nblk; ++blk) {
                const int stage = blk % STAGES;
                if (blk >= STAGES && !mbar_wait(bar_empty + 8 * stage, static_cast<uint32_t>(blk / STAGES - 1) & 1u, abort_flag)) break;
                mbar_expect_tx(bar_full + 8 * stage, Cfg::B_BYTES);
                tma_load_2d(smem_b + stage * Cfg::B_BYTES, &tmap_b, 0, (kb0 + blk) * p.tb8 + (t0 >> 3), bar_full + 8 * stage);
                // the packed tile four k-blocks ahead: its slot was read by the expansion of block
                // nb - RAW, which precedes the MMAs that just released this stage
                const int nb = blk + STAGES;
                if (nb >= RAW && nb < nblk) {
                    const int slot = nb % RAW;
                    if (!mbar_wait(bar_pk_empty + 8 * slot, static_cast<uint32_t>(nb / RAW - 1) & 1u, abort_flag)) break;
                    mbar_expect_tx(bar_pk_full + 8 * slot, kSlot);
                    bulk_load(smem_pk + slot * kSlot, v2_tiles + static_cast<size_t>(nb) * kVals2TileBytes, kVals2TileBytes, bar_pk_full + 8 * slot);
                    bulk_load(smem_pk + slot * kSlot + kVals2TileBytes, me_tiles + static_cast<size_t>(nb) * 2048, 2048, bar_pk_full + 8 * slot);
                }
            }
        }
        __syncwarp();
        cluster_wait();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && nblk > 0) {
            constexpr uint32_t idesc = make_idesc_i8(kBM, BN, true);
            bool good = true;
            for (int blk = 0; blk < nblk; ++blk) {
                const int stage = blk % STAGES;
                const uint32_t par = static_cast<uint32_t>(blk / STAGES) & 1u;
                if (!mbar_wait(bar_exp + 8 * stage, par, abort_flag) || !mbar_wait(bar_full + 8 * stage, par, abort_flag)) { good = false; break; }
                tcgen05_fence_after();
                const uint32_t e_tmem = tmem_base + static_cast<uint32_t>(Cfg::META_COL0 + 4 * stage);
                tcgen05_cp_128x128b(e_tmem, make_smem_desc(smem_e + stage * Cfg::E_BYTES, 128, 128, kSwzNone));
                const uint64_t a_desc = make_smem_desc(smem_a + stage * Cfg::A_BYTES, 16, 512, kSwz64);
                const uint64_t b_desc = make_smem_desc(smem_b + stage * Cfg::B_BYTES, 16, 1024, kSwz128);
#pragma unroll
                for (int j = 0; j < kBK / 64; ++j)
                    mma_i8_sparse(tmem_base, a_desc + static_cast<uint64_t>(2 * j), b_desc + static_cast<uint64_t>(4 * j),
                                  e_tmem + 2 * j, idesc, (blk == 0 && j == 0) ? 0u : 1u);
                tcgen05_commit(bar_empty + 8 * stage);
            }
            if (good) tcgen05_commit(bar_acc_full);
        }
        __syncwarp();
        cluster_wait();
    } else {
        // ------------------------------------------------------------------ the remaining expansions, then the scatter
        for (int blk = n_exp_pre; blk < nblk && ok; ++blk) expand_block(blk);
        const int quarter = warp & 3;
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const int f = quarter * 32 + lane;
        const bool have = nblk > 0;
        if (have && ok) {
            ok = mbar_wait(bar_acc_full, 0u, abort_flag);
            tcgen05_fence_after();
        }
        cluster_wait();
        const uint32_t my_slot = smem_red + (rank * static_cast<uint32_t>(tok_per_cta)) * (kBM * 4) + static_cast<uint32_t>(f) * 4u;
        uint32_t rr[32];
        if (have && ok) {
            tmem_ld_32x32b_x32(tmem_base + lane_base, rr);
            tmem_ld_wait();
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) rr[j] = 0u;
        }
        auto scatter = [&](auto s_const) {
            constexpr int SS = decltype(s_const)::value;
            uint32_t row_of[SS], bar_of[SS];
#pragma unroll
            for (int o = 0; o < SS; ++o) {
                row_of[o] = map_to_cta(my_slot, static_cast<uint32_t>(o));
                bar_of[o] = map_to_cta(bar_red, static_cast<uint32_t>(o));
            }
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < tile_tokens)                                       // token j: entry j / S of owner j % S
                    st_async_cluster_u32(row_of[j % SS] + static_cast<uint32_t>(j / SS) * (kBM * 4), rr[j], bar_of[j % SS]);
        };
        if (S == 2u) scatter(std::integral_constant<int, 2>{});
        else if (S == 3u) scatter(std::integral_constant<int, 3>{});
        else if (S == 4u) scatter(std::integral_constant<int, 4>{});
        else scatter(std::integral_constant<int, 8>{});
        tcgen05_fence_before();
    }
    float sc_a = 0.0f;
    if (warp >= 2) {
        const float w_scale = __ldg(p.w_scale);
        const int ja = lane * static_cast<int>(S) + static_cast<int>(rank);
        if (lane < tok_per_cta && ja < tile_tokens) sc_a = __fmul_rn(w_scale, __ldg(p.a_scale + t0 + ja));
    }
    if (warp >= 2) {
        if (!mbar_wait(bar_red, 0u, abort_flag)) ok = false;
        ok = __all_sync(0xFFFFFFFFu, ok);
        const int quarter = warp & 3;
        const int f = quarter * 32 + lane;
        const int n = mt * kBM + f;
        const float bias = p.bias ? __ldg(p.bias + n) : 0.0f;
        const int32_t* red = reinterpret_cast<const int32_t*>(smem_raw + (smem_red - smem_u32(smem_raw)));
        const bool fine = (*abort_flag == 0);
        const int n_tok = (fine && ok) ? my_tokens : 0;
        cluster_finish(S, red, tok_per_cta, n_tok, f, [&](int j, int acc) {
            const int t = t0 + j * static_cast<int>(S) + static_cast<int>(rank);
            const float sc = __shfl_sync(0xFFFFFFFFu, sc_a, j);
            if (p.acc_out) p.acc_out[static_cast<size_t>(t) * p.N + n] = acc;
            float v = __fmul_rn(static_cast<float>(acc), sc);
            if (p.bias) v = __fadd_rn(v, bias);
            if (p.out_bf16) static_cast<uint16_t*>(p.y)[static_cast<size_t>(t) * p.N + n] = static_cast<uint16_t>(f32_to_bf16_rne(v));
            else static_cast<float*>(p.y)[static_cast<size_t>(t) * p.N + n] = v;
        });
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace sbn
