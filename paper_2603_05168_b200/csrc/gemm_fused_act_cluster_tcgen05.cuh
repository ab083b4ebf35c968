// Algorithm 2's forward for few tokens in ONE kernel: per-token absmax quantisation of the bf16
// activations (Sec. 2.1) and Eq. 4.  One launch instead of two: 9.8 us against 12.8 us per BitLinear
// at T = 8 when launches are plainly serialised.  Inside a chain of programmatic dependent launches
// the separate quantiser costs only ~1.3 us and the two-kernel route is the faster one (6.4 us
// against 7.6 us): here every one of the N / 128 row tiles reads and quantises the tile's tokens
// again, and the exchange of row maxima is one more hop on the critical path.
//
// The cluster split-K kernel of gemm_splitk_cluster_tcgen05.cuh with the activation operand made
// in place: the S CTAs of a cluster share an output tile (128 features x up to 32 tokens) and
// split K, so together they see every column of the tile's tokens exactly once.
//
//   pass 1    the four epilogue warps (4 threads per token) read this CTA's K slice of x and take
//             the per-token maximum of |x| over it;
//   exchange  every CTA sends its partial maxima to all CTAs of the cluster (st.async counted on an
//             mbarrier of the receiver, as for the partial sums); the maximum over the S partials is
//             the row maximum a of Sec. 2.1 -- max is exact in any order, so d = max(a, 1e-5),
//             s_x = 127 / d and a_scale = d / 127 are bit for bit those of sbn_quant_act;
//   pass 2    the slice is read again (L1 / L2), x~ = clamp(rint(x * s_x)) goes straight into the
//             128 B-swizzled shared-memory image of the B operand, stage by stage, each stage
//             handed to the MMA thread through an mbarrier after a proxy fence;
//   then      K-loop, reduce-scatter of the partial sums and finish exactly as in the base kernel.
//
// The weights of the first stages are fetched before the dependency wait (see sbn_common.cuh);
// x, written by the kernel before this one, is only touched after it.
#pragma once

#include "quant_act.cuh"
#include "gemm_splitk_cluster_tcgen05.cuh"

namespace sbn {

struct FusedActParams {
    GemmParams g;
    const void* x_bf16;          // [T][K]
    float* a_scale_out;          // [T] or null: the per-token scales, written by the clusters of row tile 0
};

template <bool SPARSE>
struct FusedActConfig {
    static constexpr int BN = 32;
    static constexpr int A_BYTES = SPARSE ? kBM * (kBK / 2) : kBM * kBK;
    static constexpr int B_BYTES = BN * kBK;
    static constexpr int E_BYTES = SPARSE ? kBM * (kBK / 8) : 0;
    static constexpr int W_BYTES = A_BYTES + E_BYTES;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
    static constexpr int STAGES = SPARSE ? 6 : 4;
    static constexpr int REDUCE_BYTES = (BN + 4) * kBM * 4;
    static constexpr int AMAX_BYTES = 8 * BN * 4 + BN * 4;              // [S <= 8][BN] partial maxima + d[BN]
    static constexpr int BAR_BYTES = 512;
    static constexpr int META_COL0 = BN;
    static constexpr uint32_t TMEM_COLS = 64;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + REDUCE_BYTES + AMAX_BYTES + BAR_BYTES;
    static_assert(BN + 4 * STAGES <= 64, "tensor memory columns");
    static_assert(SMEM_BYTES <= 232448 / 2 - 1024, "two CTAs per SM");
};

template <bool SPARSE>
__global__ void __launch_bounds__(kSplitThreads, 2)
bitlinear_gemm_fused_act_cluster_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                        const __grid_constant__ CUtensorMap tmap_e, const FusedActParams fp) {
    using Cfg = FusedActConfig<SPARSE>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int BN = Cfg::BN;
    const GemmParams& p = fp.g;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_a + STAGES * Cfg::A_BYTES;
    const uint32_t smem_e = smem_b + STAGES * Cfg::B_BYTES;
    const uint32_t smem_red = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t smem_amax = smem_red + Cfg::REDUCE_BYTES;             // [S][BN] float bits, then d[BN]
    const uint32_t bar_base = smem_amax + Cfg::AMAX_BYTES;
    const uint32_t bar_full = bar_base;                                   // weights of a stage have landed
    const uint32_t bar_empty = bar_full + 8 * STAGES;                     // the MMAs of a stage are done
    const uint32_t bar_bq = bar_empty + 8 * STAGES;                       // a stage's activations are quantised (128 arrivals)
    const uint32_t bar_acc_full = bar_bq + 8 * STAGES;
    const uint32_t bar_red = bar_acc_full + 8;
    const uint32_t bar_amax = bar_red + 8;
    const uint32_t tmem_slot = bar_amax + 8;

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

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
            mbar_init(bar_bq + 8 * s, 128);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_red, 1);
        mbar_init(bar_amax, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // armed before any peer can send (peers send only after this CTA's cluster_arrive below)
        mbar_expect_tx(bar_red, static_cast<uint32_t>(my_tokens) * S * (kBM * 4));
        mbar_expect_tx(bar_amax, static_cast<uint32_t>(tile_tokens) * S * 4u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tcgen05_fence_before();
    }
    __syncthreads();
    tcgen05_fence_after();
    cluster_arrive();

    const int n_pre = min(STAGES, nblk);
    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmap_a);
        if constexpr (SPARSE) tma_prefetch_desc(&tmap_e);
        for (int i = 0; i < n_pre; ++i) {
            const uint32_t full = bar_full + 8 * i;
            mbar_expect_tx(full, Cfg::W_BYTES);
            const int wt = mt * p.k_blocks_total + kb0 + i;
            if constexpr (SPARSE) {
                tma_load_2d(smem_a + i * Cfg::A_BYTES, &tmap_a, 0, wt * 8, full);
                tma_load_2d(smem_e + i * Cfg::E_BYTES, &tmap_e, 0, wt * 2, full);
            } else {
                tma_load_2d(smem_a + i * Cfg::A_BYTES, &tmap_a, 0, wt * 16, full);
            }
        }
        if (nblk > n_pre) {
            const size_t wt0 = static_cast<size_t>(mt) * p.k_blocks_total + kb0 + n_pre;
            prefetch_l2_bulk(static_cast<const char*>(p.w_vals) + wt0 * p.w_tile_bytes, static_cast<uint32_t>((nblk - n_pre) * p.w_tile_bytes));
            if (p.w_meta) prefetch_l2_bulk(static_cast<const char*>(p.w_meta) + wt0 * 2048, static_cast<uint32_t>((nblk - n_pre) * 2048));
        }
    }
    pdl_wait();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    bool ok = true;
    if (warp == 0) {
        // ------------------------------------------------------------------ producer: the later weight stages
        if (lane == 0) {
            for (int blk = n_pre; blk < nblk; ++blk) {
                const int stage = blk % STAGES;
                if (!mbar_wait(bar_empty + 8 * stage, static_cast<uint32_t>(blk / STAGES - 1) & 1u, abort_flag)) break;
                const uint32_t full = bar_full + 8 * stage;
                mbar_expect_tx(full, Cfg::W_BYTES);
                const int wt = mt * p.k_blocks_total + kb0 + blk;
                if constexpr (SPARSE) {
                    tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 8, full);
                    tma_load_2d(smem_e + stage * Cfg::E_BYTES, &tmap_e, 0, wt * 2, full);
                } else {
                    tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 16, full);
                }
            }
        }
        __syncwarp();
        cluster_wait();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && nblk > 0) {
            constexpr uint32_t idesc = make_idesc_i8(kBM, BN, SPARSE);
            bool good = true;
            for (int blk = 0; blk < nblk; ++blk) {
                const int stage = blk % STAGES;
                const uint32_t par = static_cast<uint32_t>(blk / STAGES) & 1u;
                if (!mbar_wait(bar_full + 8 * stage, par, abort_flag) || !mbar_wait(bar_bq + 8 * stage, par, abort_flag)) { good = false; break; }
                tcgen05_fence_after();
                const uint32_t a_addr = smem_a + stage * Cfg::A_BYTES;
                const uint32_t b_addr = smem_b + stage * Cfg::B_BYTES;
                const uint32_t first = (blk == 0) ? 0u : 1u;
                if constexpr (SPARSE) {
                    const uint32_t e_tmem = tmem_base + static_cast<uint32_t>(Cfg::META_COL0 + 4 * stage);
                    tcgen05_cp_128x128b(e_tmem, make_smem_desc(smem_e + stage * Cfg::E_BYTES, 128, 128, kSwzNone));
                    const uint64_t a_desc = make_smem_desc(a_addr, 16, 512, kSwz64);
                    const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
#pragma unroll
                    for (int j = 0; j < kBK / 64; ++j)
                        mma_i8_sparse(tmem_base, a_desc + static_cast<uint64_t>(2 * j), b_desc + static_cast<uint64_t>(4 * j),
                                      e_tmem + 2 * j, idesc, j == 0 ? first : 1u);
                } else {
                    const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024, kSwz128);
                    const uint64_t b_desc = make_smem_desc(b_addr, 16, 1024, kSwz128);
#pragma unroll
                    for (int j = 0; j < kBK / 32; ++j)
                        mma_i8_dense(tmem_base, a_desc + static_cast<uint64_t>(2 * j), b_desc + static_cast<uint64_t>(2 * j),
                                     idesc, j == 0 ? first : 1u);
                }
                tcgen05_commit(bar_empty + 8 * stage);
            }
            if (good) tcgen05_commit(bar_acc_full);
        }
        __syncwarp();
        cluster_wait();
    } else {
        // ------------------------------------------------------------------ quantise the activations, then the epilogue
        const uint32_t tix = threadIdx.x - 64;
        const int tok = static_cast<int>(tix >> 2);                       // token of the tile: 4 threads each
        const uint32_t sub = tix & 3u;                                    // 32 of a k-block's 128 columns
        const bool real = tok < tile_tokens;
        const uint4* xrow = reinterpret_cast<const uint4*>(static_cast<const char*>(fp.x_bf16) +
                                                           (static_cast<size_t>(t0 + tok) * p.K + static_cast<size_t>(kb0) * kBK + sub * 32u) * 2u);
        // pass 1: maximum of |x| over this CTA's slice (bit patterns of non-negative bf16 order like integers)
        uint32_t pm = 0u;
        if (real) {
            int blk = 0;
            for (; blk + 4 <= nblk; blk += 4) {                          // 16 independent loads in flight
                uint4 v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = __ldg(xrow + (blk + (i >> 2)) * 16 + (i & 3));
#pragma unroll
                for (int i = 0; i < 16; ++i) pm = absmax8_packed(v[i], pm);
            }
            for (; blk < nblk; ++blk) {
#pragma unroll
                for (int i = 0; i < 4; ++i) pm = absmax8_packed(__ldg(xrow + blk * 16 + i), pm);
            }
        }
        uint32_t mbits = max(pm >> 16, pm & 0xFFFFu) << 16;               // fp32 bits of the partial maximum
        mbits = max(mbits, __shfl_xor_sync(0xFFFFFFFFu, mbits, 1));
        mbits = max(mbits, __shfl_xor_sync(0xFFFFFFFFu, mbits, 2));
        cluster_wait();                                                   // all peers have started
        if (real && sub == 0u) {
            const uint32_t slot = smem_amax + (rank * BN + static_cast<uint32_t>(tok)) * 4u;
            for (uint32_t o = 0; o < S; ++o) st_async_cluster_u32(map_to_cta(slot, o), mbits, map_to_cta(bar_amax, o));
        }
        if (!mbar_wait(bar_amax, 0u, abort_flag)) ok = false;
        float s_x = 0.0f;
        if (real) {
            uint32_t m = 0u;
            for (uint32_t s2 = 0; s2 < S; ++s2) {
                uint32_t v;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_amax + (s2 * BN + static_cast<uint32_t>(tok)) * 4u));
                m = max(m, v);
            }
            const float d = fmaxf(__uint_as_float(m), kEps);
            s_x = __fdiv_rn(127.0f, d);
            if (sub == 0u) {
                const float a_sc = __fdiv_rn(d, 127.0f);
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_amax + (8u * BN + static_cast<uint32_t>(tok)) * 4u), "f"(a_sc) : "memory");
                if (fp.a_scale_out && mt == 0 && rank == 0) fp.a_scale_out[t0 + tok] = a_sc;
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");                    // the scales are read by other threads in the finish
        // pass 2: x~ into the B image of every stage (row = token, 128 B, 16 B chunks XOR-ed with row % 8)
        const uint32_t brow = (static_cast<uint32_t>(tok) >> 3) * 1024u + (static_cast<uint32_t>(tok) & 7u) * 128u;
        // (L1 is too small next to two CTAs' shared memory to keep pass 1's lines: this pass reads from L2
        // again, one k-block ahead of the one being written)
        uint4 nxt[4] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
        if (real && nblk > 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) nxt[i] = __ldg(xrow + i);
        }
        for (int blk = 0; blk < nblk && ok; ++blk) {
            const int stage = blk % STAGES;
            uint4 cur[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
            if (real && blk + 1 < nblk) {
#pragma unroll
                for (int i = 0; i < 4; ++i) nxt[i] = __ldg(xrow + (blk + 1) * 16 + i);
            }
            if (blk >= STAGES && !mbar_wait(bar_empty + 8 * stage, static_cast<uint32_t>(blk / STAGES - 1) & 1u, abort_flag)) { ok = false; break; }
            uint32_t c[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                c[2 * i] = quant_pair2(cur[i].x, cur[i].y, s_x);          // padding tokens: zeros in, zeros out
                c[2 * i + 1] = quant_pair2(cur[i].z, cur[i].w, s_x);
            }
            const uint32_t base = smem_b + stage * Cfg::B_BYTES + brow;
            const uint32_t r7 = static_cast<uint32_t>(tok) & 7u;
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(base + (((2u * sub) ^ r7) << 4)), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]) : "memory");
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(base + (((2u * sub + 1u) ^ r7) << 4)), "r"(c[4]), "r"(c[5]), "r"(c[6]), "r"(c[7]) : "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(bar_bq + 8 * stage);
        }

        // ------------------------------------------------------------------ epilogue, part 1: scatter
        const int quarter = warp & 3;
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const int f = quarter * 32 + lane;
        const bool have = nblk > 0;
        if (have && ok) {
            ok = mbar_wait(bar_acc_full, 0u, abort_flag);
            tcgen05_fence_after();
        }
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
                if (j < tile_tokens)
                    st_async_cluster_u32(row_of[j % SS] + static_cast<uint32_t>(j / SS) * (kBM * 4), rr[j], bar_of[j % SS]);
        };
        if (S == 2u) scatter(std::integral_constant<int, 2>{});
        else if (S == 3u) scatter(std::integral_constant<int, 3>{});
        else if (S == 4u) scatter(std::integral_constant<int, 4>{});
        else scatter(std::integral_constant<int, 8>{});
        tcgen05_fence_before();

        // ------------------------------------------------------------------ epilogue, part 2: finish my tokens
        if (!mbar_wait(bar_red, 0u, abort_flag)) ok = false;
        ok = __all_sync(0xFFFFFFFFu, ok);
        const int n = mt * kBM + f;
        const float w_scale = __ldg(p.w_scale);
        const float bias = p.bias ? __ldg(p.bias + n) : 0.0f;
        const int32_t* red = reinterpret_cast<const int32_t*>(smem_raw + (smem_red - smem_u32(smem_raw)));
        const float* a_sc = reinterpret_cast<const float*>(smem_raw + (smem_amax + 8u * BN * 4u - smem_u32(smem_raw)));
        const bool fine = (*abort_flag == 0);
        const int n_tok = (fine && ok) ? my_tokens : 0;
        cluster_finish(S, red, tok_per_cta, n_tok, f, [&](int j, int acc) {
            const int tl = j * static_cast<int>(S) + static_cast<int>(rank);          // token inside the tile
            const float sc = __fmul_rn(w_scale, a_sc[tl]);
            const size_t o = static_cast<size_t>(t0 + tl) * p.N + n;
            if (p.acc_out) p.acc_out[o] = acc;
            float v = __fmul_rn(static_cast<float>(acc), sc);
            if (p.bias) v = __fadd_rn(v, bias);
            if (p.out_bf16) static_cast<uint16_t*>(p.y)[o] = static_cast<uint16_t>(f32_to_bf16_rne(v));
            else static_cast<float*>(p.y)[o] = v;
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
