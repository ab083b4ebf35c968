// Eq. 4 for few tokens: split-K inside a thread-block cluster.
//
// With T up to a few hundred there are only N/128 x ceil(T/BN) output tiles -- far fewer than SMs --
// and a CTA that walks the whole K of its tile is bound by what ONE SM can pull out of L2
// (~100 GB/s: 18 KB per 128 columns -> 0.23 us each).  Splitting K over CTAs puts more SMs on the
// weight stream; the partial accumulators then have to be added.  Through global memory that is
// one int32 atomic per output element and slice, which costs more than the K-loop it saves once
// T reaches 64.  Here the S CTAs that share an output tile form a CLUSTER and add their partial
// accumulators through distributed shared memory:
//
//   CTA r of the cluster   k-blocks [r q, min((r+1) q, K/128)),  q = ceil(K/128 / S)
//   mainloop               as in the single-CTA kernel (TMA producer warp, MMA issuer warp,
//                          metadata through tcgen05.cp, one accumulator in TMEM)
//   reduce-scatter         CTA r owns the tokens j with j % S == r (interleaved, so that a tile with
//                          few real tokens still spreads them over all CTAs); each epilogue thread
//                          (one output feature = one TMEM lane) writes its partial sums of every
//                          REAL token j straight into the shared memory of the CTA that owns j
//                          with st.async, slot [r]; padding tokens are skipped.  Every such store
//                          counts its 4 bytes on an mbarrier of the OWNER, which expects exactly
//                          (its tokens) x S x 128 x 4 bytes: no cluster-wide barrier after the
//                          scatter, each CTA goes on as soon as ITS partials are complete
//   finish                 every CTA adds the S partials of its tokens, applies s = w_scale *
//                          a_scale[t] (+ bias) and stores y (and the int32 dump when asked for)
//
// No scratch in global memory, no atomics, nothing to keep zeroed.  A CTA leaves only after all
// bytes addressed to it have arrived, and nothing is addressed to a CTA that owns no real token,
// so no store ever targets shared memory of a CTA that has exited.  All mbarrier waits are bounded.
#pragma once

#include <type_traits>

#include "gemm_pair_tcgen05.cuh"

namespace sbn {

constexpr int kSplitThreads = 192;        // warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 epilogue
constexpr int kSplitMaxCluster = 8;

template <bool SPARSE, int BN>
struct SplitConfig {
    static constexpr int A_BYTES = SPARSE ? kBM * (kBK / 2) : kBM * kBK;
    static constexpr int B_BYTES = BN * kBK;
    static constexpr int E_BYTES = SPARSE ? kBM * (kBK / 8) : 0;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
    // BN <= 64: few enough stages that TWO CTAs fit on an SM (< 113 KB each), so the CTAs of the next
    // launch of a decode loop are resident -- and already pulling their weights -- while this one
    // reduces and finishes.  A stage that is filled before the dependency wait costs nothing, one
    // that has to be refilled costs an L2 round trip on the critical path: the 32-token tile keeps
    // six (sparse) stages, enough for the whole K slice of a CTA at the usual sizes.
    static constexpr int STAGES = (BN == 32) ? (SPARSE ? 6 : 4) : (BN == 64) ? (SPARSE ? 4 : 3) : (SPARSE ? 6 : 4);
    static constexpr int CTAS_PER_SM = (BN <= 64) ? 2 : 1;
    static constexpr int REDUCE_BYTES = (BN + 4) * kBM * 4;    // [S][ceil(BN/S) tokens][128 features] int32, S in {2, 3, 4, 8}
    static constexpr int META_COL0 = BN;                        // metadata columns above the accumulator
    static constexpr uint32_t TMEM_COLS = (BN + 4 * STAGES <= 64) ? 64 : (BN + 4 * STAGES <= 128 ? 128 : 256);
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + REDUCE_BYTES + kBarrierBytes;
    static_assert(SMEM_BYTES <= 232448 / CTAS_PER_SM - 1024 * (CTAS_PER_SM - 1), "shared memory overflow");
    static_assert(BN % 32 == 0 && BN <= 128, "token tile");
};

// 4-byte store into a peer's shared memory that counts its bytes on an mbarrier of that peer.
__device__ __forceinline__ void st_async_cluster_u32(uint32_t cluster_addr, uint32_t v, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "r"(v), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}

// Adds the S partial sums of each of this CTA's n_tok tokens (buffer [S][tok_per_cta][128] int32, this
// thread's feature f) and hands (local token index, sum) to `emit`.  Four tokens at a time with S known
// at compile time: 4 * S independent loads in flight -- the one-token-at-a-time loop with a run-time S
// was a chain of shared-memory latencies, 0.12 us per token.
template <int SS, typename Emit>
__device__ __forceinline__ void cluster_finish_tokens(const int32_t* red, int tok_per_cta, int n_tok, int f, Emit emit) {
    int j = 0;
    for (; j + 4 <= n_tok; j += 4) {
        int acc[4] = {0, 0, 0, 0};
#pragma unroll
        for (int s2 = 0; s2 < SS; ++s2)
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] += red[(s2 * tok_per_cta + j + u) * kBM + f];
#pragma unroll
        for (int u = 0; u < 4; ++u) emit(j + u, acc[u]);
    }
    for (; j < n_tok; ++j) {
        int acc = 0;
#pragma unroll
        for (int s2 = 0; s2 < SS; ++s2) acc += red[(s2 * tok_per_cta + j) * kBM + f];
        emit(j, acc);
    }
}
template <typename Emit>
__device__ __forceinline__ void cluster_finish(uint32_t S, const int32_t* red, int tok_per_cta, int n_tok, int f, Emit emit) {
    if (S == 2u) cluster_finish_tokens<2>(red, tok_per_cta, n_tok, f, emit);
    else if (S == 3u) cluster_finish_tokens<3>(red, tok_per_cta, n_tok, f, emit);
    else if (S == 4u) cluster_finish_tokens<4>(red, tok_per_cta, n_tok, f, emit);
    else cluster_finish_tokens<8>(red, tok_per_cta, n_tok, f, emit);
}

template <bool SPARSE, int BN>
__global__ void __launch_bounds__(kSplitThreads, SplitConfig<SPARSE, BN>::CTAS_PER_SM)
bitlinear_gemm_splitk_cluster_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                     const __grid_constant__ CUtensorMap tmap_b,
                                     const __grid_constant__ CUtensorMap tmap_e,
                                     const GemmParams p) {
    using Cfg = SplitConfig<SPARSE, BN>;
    constexpr int STAGES = Cfg::STAGES;

    extern __shared__ uint8_t smem_raw[];
    // 1 KB alignment: required by the 128 B swizzle atoms; the offset is the same in every CTA of
    // the cluster (same kernel, same static shared memory), so peers' buffers sit at the same offset
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_a = smem_base;
    const uint32_t smem_b = smem_a + STAGES * Cfg::A_BYTES;
    const uint32_t smem_e = smem_b + STAGES * Cfg::B_BYTES;
    const uint32_t smem_red = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = smem_red + Cfg::REDUCE_BYTES;
    const uint32_t bar_full = bar_base;
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_acc_full = bar_empty + 8 * STAGES;
    const uint32_t bar_red = bar_acc_full + 8;               // counts the bytes of partial sums sent to this CTA
    const uint32_t tmem_slot = bar_red + 8;

    __shared__ int s_abort;
    volatile int* abort_flag = &s_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t S = cluster_nctarank();
    const int tile = blockIdx.x / static_cast<int>(S);          // clusters are consecutive blocks
    const int tiles_m = p.N / kBM;
    const int mt = tile % tiles_m;
    const int tt = tile / tiles_m;
    const int t0 = tt * BN;
    const int q = (p.k_blocks_total + static_cast<int>(S) - 1) / static_cast<int>(S);
    const int kb0 = min(p.k_blocks_total, static_cast<int>(rank) * q);
    const int kb1 = min(p.k_blocks_total, kb0 + q);
    const int tok_per_cta = (BN + static_cast<int>(S) - 1) / static_cast<int>(S);   // S is 2, 3, 4 or 8 (host's duty)
    const int tile_tokens = min(BN, p.T - t0);                  // real tokens of this tile
    // my tokens: rank, rank + S, ... below tile_tokens
    const int my_tokens = max(0, (tile_tokens - static_cast<int>(rank) + static_cast<int>(S) - 1) / static_cast<int>(S));

    pdl_launch_dependents();             // lets the kernels after this one become resident as early as possible
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_red, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // armed before any peer can send: peers scatter only after this CTA's cluster_arrive below
        mbar_expect_tx(bar_red, static_cast<uint32_t>(my_tokens) * S * (kBM * 4));
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tcgen05_fence_before();
    }
    __syncthreads();
    tcgen05_fence_after();
    // a peer's shared memory may only be written once that CTA has started: every thread arrives
    // here and waits just before the scatter, so the barrier costs nothing on the way in
    cluster_arrive();
    // The weights of the first stages are fetched while the previous kernel of the stream is still
    // finishing.  This is safe because no kernel that WRITES packed weights signals its dependents
    // early (see sbn_common.cuh): a kernel that is running implies every earlier weight producer
    // has completed.  The activations (written by the kernel right before this one) wait.
    const int n_pre = min(STAGES, kb1 - kb0);
    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
        if constexpr (SPARSE) tma_prefetch_desc(&tmap_e);
        for (int i = 0; i < n_pre; ++i) {
            const uint32_t full = bar_full + 8 * i;
            mbar_expect_tx(full, Cfg::STAGE_BYTES);
            const int wt = mt * p.k_blocks_total + kb0 + i;
            if constexpr (SPARSE) {
                tma_load_2d(smem_a + i * Cfg::A_BYTES, &tmap_a, 0, wt * 8, full);
                tma_load_2d(smem_e + i * Cfg::E_BYTES, &tmap_e, 0, wt * 2, full);
            } else {
                tma_load_2d(smem_a + i * Cfg::A_BYTES, &tmap_a, 0, wt * 16, full);
            }
        }
        // the rest of this CTA's slice goes to L2 (the point of coherence: nothing can go stale there)
        if (kb1 - kb0 > n_pre) {
            const size_t wt0 = static_cast<size_t>(mt) * p.k_blocks_total + kb0 + n_pre;
            prefetch_l2_bulk(static_cast<const char*>(p.w_vals) + wt0 * p.w_tile_bytes, static_cast<uint32_t>((kb1 - kb0 - n_pre) * p.w_tile_bytes));
            if (p.w_meta) prefetch_l2_bulk(static_cast<const char*>(p.w_meta) + wt0 * 2048, static_cast<uint32_t>((kb1 - kb0 - n_pre) * 2048));
        }
    }
    pdl_wait();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    bool ok = true;
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && !p.test_skip_loads) {
            int stage = 0;
            uint32_t phase = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                const uint32_t full = bar_full + 8 * stage;
                if (kb - kb0 >= n_pre) {                                 // the first n_pre stages got their weights above
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) break;
                    mbar_expect_tx(full, Cfg::STAGE_BYTES);
                    const int wt = mt * p.k_blocks_total + kb;            // weight tile index
                    if constexpr (SPARSE) {
                        tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 8, full);
                        tma_load_2d(smem_e + stage * Cfg::E_BYTES, &tmap_e, 0, wt * 2, full);
                    } else {
                        tma_load_2d(smem_a + stage * Cfg::A_BYTES, &tmap_a, 0, wt * 16, full);
                    }
                }
                tma_load_2d(smem_b + stage * Cfg::B_BYTES, &tmap_b, 0, kb * p.tb8 + (t0 >> 3), full);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
        cluster_wait();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && kb1 > kb0) {
            constexpr uint32_t idesc = make_idesc_i8(kBM, BN, SPARSE);
            int stage = 0;
            uint32_t phase = 0;
            bool good = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { good = false; break; }
                tcgen05_fence_after();
                const uint32_t a_addr = smem_a + stage * Cfg::A_BYTES;
                const uint32_t b_addr = smem_b + stage * Cfg::B_BYTES;
                const uint32_t first = (kb == kb0) ? 0u : 1u;
                if constexpr (SPARSE) {
                    const uint32_t e_tmem = tmem_base + static_cast<uint32_t>(Cfg::META_COL0 + 4 * stage);
                    const uint64_t e_desc = make_smem_desc(smem_e + stage * Cfg::E_BYTES, 128, 128, kSwzNone);
                    tcgen05_cp_128x128b(e_tmem, e_desc);
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
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (good) tcgen05_commit(bar_acc_full);
        }
        __syncwarp();
        cluster_wait();
    } else {
        // ------------------------------------------------------------------ epilogue, part 1: scatter
        const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const int f = quarter * 32 + lane;                // feature inside the tile
        const bool have = kb1 > kb0;                      // an empty K slice contributes zeros
        if (have) {
            ok = mbar_wait(bar_acc_full, 0u, abort_flag);
            tcgen05_fence_after();
        }
        cluster_wait();                                   // all peers have started
        // slot [rank][token / S][feature] in the buffer of the owner, CTA token % S
        const uint32_t my_slot = smem_red + (rank * static_cast<uint32_t>(tok_per_cta)) * (kBM * 4) + static_cast<uint32_t>(f) * 4u;
        auto scatter = [&](auto s_const) {
            constexpr int SS = decltype(s_const)::value;                  // compile-time: token / S and token % S cost nothing
#pragma unroll 1
            for (int c = 0; c * 32 < tile_tokens; ++c) {
                uint32_t r[32];
                if (have && ok) {
                    tmem_ld_32x32b_x32(tmem_base + lane_base + static_cast<uint32_t>(c * 32), r);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                uint32_t row_of[SS], bar_of[SS];
#pragma unroll
                for (int o = 0; o < SS; ++o) {
                    row_of[o] = map_to_cta(my_slot, static_cast<uint32_t>(o));
                    bar_of[o] = map_to_cta(bar_red, static_cast<uint32_t>(o));
                }
                // BN is a multiple of 32, but 32 is not a multiple of 3: token = c * 32 + j
                const int base_owner = (c * 32) % SS, base_local = (c * 32) / SS;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int tok = c * 32 + j;
                    if (tok < tile_tokens) {                               // warp-uniform
                        if constexpr ((32 % SS) == 0) {
                            st_async_cluster_u32(row_of[j % SS] + static_cast<uint32_t>(base_local + j / SS) * (kBM * 4), r[j], bar_of[j % SS]);
                        } else {
                            const int o = (base_owner + j) % SS, l = (c * 32 + j) / SS;
                            uint32_t ra = row_of[0], ba = bar_of[0];
#pragma unroll
                            for (int k = 1; k < SS; ++k)
                                if (o == k) { ra = row_of[k]; ba = bar_of[k]; }
                            st_async_cluster_u32(ra + static_cast<uint32_t>(l) * (kBM * 4), r[j], ba);
                        }
                    }
                }
            }
        };
        if (S == 2u) scatter(std::integral_constant<int, 2>{});
        else if (S == 3u) scatter(std::integral_constant<int, 3>{});
        else if (S == 4u) scatter(std::integral_constant<int, 4>{});
        else scatter(std::integral_constant<int, 8>{});
        tcgen05_fence_before();
    }
    // s of Eq. 4 for the tokens this CTA finishes, fetched before the barrier (lane l: its l-th and
    // (l + 32)-th token) so that the finishing loop has no global load to wait for
    float sc_a = 0.0f, sc_b = 0.0f;
    if (warp >= 2) {
        const float w_scale = __ldg(p.w_scale);
        const int ja = lane * static_cast<int>(S) + static_cast<int>(rank);          // token inside the tile
        const int jb = (lane + 32) * static_cast<int>(S) + static_cast<int>(rank);
        if (lane < tok_per_cta && ja < tile_tokens) sc_a = __fmul_rn(w_scale, __ldg(p.a_scale + t0 + ja));
        if (lane + 32 < tok_per_cta && jb < tile_tokens) sc_b = __fmul_rn(w_scale, __ldg(p.a_scale + t0 + jb));
    }

    if (warp >= 2) {
        // all partial sums addressed to this CTA have landed (the barrier's phase completes with the
        // last byte; its completion makes the asynchronous stores visible to the waiting threads)
        if (!mbar_wait(bar_red, 0u, abort_flag)) ok = false;
        ok = __all_sync(0xFFFFFFFFu, ok);                 // the loop below shuffles: one decision per warp
        // ------------------------------------------------------------------ epilogue, part 2: finish my tokens
        const int quarter = warp & 3;
        const int f = quarter * 32 + lane;
        const int n = mt * kBM + f;
        const float bias = p.bias ? __ldg(p.bias + n) : 0.0f;
        const int32_t* red = reinterpret_cast<const int32_t*>(smem_raw + (smem_red - smem_u32(smem_raw)));
        const bool fine = (*abort_flag == 0);
        const int n_tok = (fine && ok) ? my_tokens : 0;
        cluster_finish(S, red, tok_per_cta, n_tok, f, [&](int j, int acc) {
            const int t = t0 + j * static_cast<int>(S) + static_cast<int>(rank);
            const float sc = __shfl_sync(0xFFFFFFFFu, j < 32 ? sc_a : sc_b, j & 31);
            if (p.acc_out) p.acc_out[static_cast<size_t>(t) * p.N + n] = acc;
            float v = __fmul_rn(static_cast<float>(acc), sc);
            if (p.bias) v = __fadd_rn(v, bias);
            if (p.out_bf16) static_cast<uint16_t*>(p.y)[static_cast<size_t>(t) * p.N + n] = static_cast<uint16_t>(f32_to_bf16_rne(v));
            else static_cast<float*>(p.y)[static_cast<size_t>(t) * p.N + n] = v;
        });
    }

    // teardown
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace sbn
