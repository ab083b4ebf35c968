// libsbn: the C ABI declared in include/sbn.h.  Host side only validates arguments, encodes TMA
// tensor maps and enqueues kernels on the caller's stream; every step of the path runs in the
// kernels of this translation unit.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <mutex>
#include <vector>

#include "sbn.h"
#include "sbn_common.cuh"
#include "quant_act.cuh"
#include "norm_quant_act.cuh"
#include "quantize_mask_pack.cuh"
#include "quantize_mask_pack68.cuh"
#include "quantize_mask_pack_stream.cuh"
#include "canonical_layout.cuh"
#include "gemm_tcgen05.cuh"
#include "gemm_pair_tcgen05.cuh"
#include "gemm_splitk_cluster_tcgen05.cuh"
#include "gemm_packed_cluster_tcgen05.cuh"
#include "gemm_fused_act_cluster_tcgen05.cuh"
#include "backward_prep.cuh"
#include "gemm_bf16_pair_tcgen05.cuh"

namespace sbn {

// ------------------------------------------------------------------------------------------------
// host state
// ------------------------------------------------------------------------------------------------
static int g_force_token_tile = 0;
static int g_force_split_k = 0;            // > 0: global-atomics split-K factor; -2, -4, -8: cluster split-K of that size
static bool g_allow_cluster = true;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess) {
            fn = reinterpret_cast<EncodeTiledFn>(p);
        }
    });
    return fn;
}

// 3-D view [d2][d1][1 KB] of tiled operand data (1 KB rows of 128 x uint64); box {1 KB, b1, b2}.
static bool encode_3d_1k(CUtensorMap* map, const void* base, uint64_t d1, uint64_t d2, uint32_t b1, uint32_t b2) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || b1 == 0 || b1 > 256 || b2 == 0 || b2 > 256) return false;
    cuuint64_t dims[3] = {128, d1, d2};
    cuuint64_t strides[2] = {1024, 1024 * d1};
    cuuint32_t box[3] = {128, b1, b2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 3, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 2-D row-major output tensor y [T][N] (fp32 or bf16) with a 32-feature x box_tokens box.
static bool encode_2d_out(CUtensorMap* map, const void* base, uint64_t N, uint64_t T, bool bf16,
                          uint32_t box_tokens, uint32_t box_features = 32) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const uint64_t es = bf16 ? 2 : 4;
    cuuint64_t dims[2] = {N, T};
    cuuint64_t strides[1] = {N * es};
    cuuint32_t box[2] = {box_features, box_tokens};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Flat array of tiled operand data viewed as rows of 1 KB (128 x uint64); box = box_rows rows.
static bool encode_flat_1k(CUtensorMap* map, const void* base, uint64_t total_bytes, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || total_bytes % 1024 != 0) return false;
    cuuint64_t dims[2] = {128, total_bytes / 1024};
    cuuint64_t strides[1] = {1024};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Row-major bf16 matrix [rows][ld] of which `inner` columns are valid, fetched in boxes of 64 columns x
// box_rows rows with the 128-byte swizzle: the box lands in shared memory as the K-major operand image.
static bool encode_2d_bf16_sw128(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || box_rows == 0 || box_rows > 256 || (ld * 2) % 16 != 0) return false;
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

static inline bool misaligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0;
}

static inline int pick_token_tile(int T) {
    if (g_force_token_tile == 64 || g_force_token_tile == 128 || g_force_token_tile == 256)
        return g_force_token_tile;
    if (T <= 64) return 64;
    return 128;
}

static inline int pick_split_k(int T, int N, int K, int bn) {
    const int kblocks = K / kBK;
    int want = 1;
    if (g_force_split_k > 0) {
        want = g_force_split_k;
    } else {
        const int tiles = (N / kBM) * ((T + bn - 1) / bn);
        // weight-streaming regime: too few tiles to cover the SMs -> split K
        if (tiles * 2 <= kNumSMs) {
            want = kNumSMs / tiles;
        }
    }
    if (want > kblocks) want = kblocks;
    while (want > 1 && kblocks % want != 0) --want;
    return want < 1 ? 1 : want;
}

static size_t split_acc_bytes(int T, int N) {
    return (static_cast<size_t>(T) * N * sizeof(int32_t) + 255) & ~static_cast<size_t>(255);
}

struct GemmPlan {
    bool pair;      // CTA-pair kernel (two M-tiles per CTA) or single-CTA tiles
    int bn;         // token tile
    int splits;     // split-K factor through global atomics (single-CTA kernel only)
    int cluster;    // > 1: split-K inside clusters of this many CTAs (reduction in shared memory)
    int mt = 2;     // CTA-pair kernel: M-tiles per CTA (2: 512-feature tiles; 1: 256-feature tiles, double-buffered accumulators)
};
static GemmPlan plan_gemm(bool sparse, int T, int N, int K);

static size_t gemm_workspace_bytes(bool sparse, int T, int N, int K) {
    // split-K scratch: int32 [T][N] + one counter per output tile; only the small-T regime splits
    const GemmPlan plan = plan_gemm(sparse, T, N, K);
    if (!plan.pair && plan.splits > 1)
        return split_acc_bytes(T, N) + static_cast<size_t>(N / kBM) * ((T + plan.bn - 1) / plan.bn) * sizeof(unsigned int);
    return 0;
}

template <bool SPARSE, int BN>
static sbn_status launch_gemm_cfg(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& te,
                                  const CUtensorMap& ty, const GemmParams& p, cudaStream_t stream) {
    using Cfg = GemmConfig<SPARSE, BN>;
    auto kernel = bitlinear_gemm_kernel<SPARSE, BN>;
    if (!ensure_dynamic_smem<bitlinear_gemm_kernel<SPARSE, BN>>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
    const int tiles = (p.N / kBM) * ((p.T + BN - 1) / BN) * p.k_splits;
    const int grid = tiles < kNumSMs ? tiles : kNumSMs;
    const cudaError_t err = launch_kernel(kernel, dim3(grid), dim3(kGemmThreads), Cfg::SMEM_BYTES, stream, ta, tb, te, ty, p);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

// ---- CTA-pair kernel (large T) -------------------------------------------------------------------
// Token-tile width for the pair kernel: a small cost model of (operand ingest | MMA rate) per unit
// of K, the accumulator drain per tile, and the number of waves over the 74 CTA pairs.
static int pick_pair_bn(bool sparse, int T, int N, int K) {
    if (g_force_token_tile < 0) {
        int bn = -g_force_token_tile;
        const int cap = sparse ? kPairMaxBnSparse : kPairMaxBnDense;
        bn = (bn / 16) * 16;
        if (bn < 32) bn = 32;
        if (bn > cap) bn = cap;
        return bn;
    }
    const int cap = sparse ? kPairMaxBnSparse : kPairMaxBnDense;
    const double mac_rate = sparse ? 16384.0 : 8192.0;          // MAC / clk / SM
    const double ingest = 64.0;                                  // B / clk / SM
    const int full_m = N / 512, rem_m = (N % 512) ? 1 : 0;
    int best = 128;
    double best_cost = 1e300;
    for (int bn = 64; bn <= cap; bn += 16) {
        const int tt = (T + bn - 1) / bn;
        auto tile_clk = [&](int mtiles) {
            const double a_bytes = sparse ? 72.0 : 128.0;
            const double bytes = mtiles * a_bytes + bn / 2.0;
            const double macs = mtiles * 128.0 * bn;
            const double per_k = std::max(bytes / ingest, macs / mac_rate);
            return per_k * K + 12.0 * bn + 600.0;                // + drain and tile turnaround
        };
        // greedy waves: full tiles first, then the half tiles
        const double work = static_cast<double>(full_m) * tt * tile_clk(2) + static_cast<double>(rem_m) * tt * tile_clk(1);
        const long tiles = static_cast<long>(full_m + rem_m) * tt;
        const long waves = (tiles + 73) / 74;
        const double balanced = work / 74.0;
        const double quantised = static_cast<double>(waves) * tile_clk(2);
        const double cost = std::max(balanced, 0.5 * (balanced + quantised));
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

template <bool SPARSE, int MT>
static sbn_status launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& te,
                              const PairParams& pp, cudaStream_t stream) {
    using Cfg = PairConfig<SPARSE, MT>;
    auto kernel = bitlinear_gemm_pair_kernel<SPARSE, MT>;
    if (!ensure_dynamic_smem<bitlinear_gemm_pair_kernel<SPARSE, MT>>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
    const int tiles = ((pp.g.N + 256 * MT - 1) / (256 * MT)) * ((pp.g.T + pp.bn - 1) / pp.bn);
    const int pairs = tiles < kNumSMs / 2 ? tiles : kNumSMs / 2;
    const cudaError_t err = launch_kernel(kernel, dim3(2 * pairs), dim3(kPairThreads), Cfg::SMEM_BYTES, stream, ta, tb, te, pp);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

// Which kernel, which token tile, whether to split K: a small model of the measured times (us).
//   single-CTA kernel   F(bn) + waves * (K/128 / splits) * c(bn)  [+ split-K: 1 + 8e-6 per atomic]
//                       F = 3.0 + 0.02 bn (prologue + last epilogue), c = 0.23 (bn = 64) | 0.27 (128) | 0.49 (256)
//   CTA-pair kernel     4.3 + 0.02 bn + waves * (K/128 * 0.31 + 2.5 (exposed drain)); dense K-loop x 1.65;
//                       with one M-tile per CTA: 4.3 + 0.02 bn + waves * K/128 * 0.205 (dense 0.29)
// waves over 148 CTAs resp. 74 pairs.  Small problems are latency-bound and favour many small
// single-CTA tiles; large ones favour the pair kernel's operand reuse.  K is split only when the
// tiles cannot fill the machine and the int32 atomics cost less than the K-loop they save.
static GemmPlan plan_gemm(bool sparse, int T, int N, int K) {
    GemmPlan best = {false, 64, 1, 0};
    const int kb = K / kBK;
    const int rows = N / kBM;
    if (g_force_token_tile < 0) {                               // diagnostics: the pair kernel as told (split_k 1 = one M-tile per CTA)
        GemmPlan g{true, pick_pair_bn(sparse, T, N, K), 1, 0};
        g.mt = g_force_split_k == 1 ? 1 : 2;
        return g;
    }
    if (g_force_split_k < 0) {                                  // diagnostics: cluster split-K as told
        int S = -g_force_split_k;
        S = S >= 8 ? 8 : (S >= 4 ? 4 : (S == 3 ? 3 : 2));
        while (S > 1 && S > K / kBK) --S;
        if (S > 4 && S < 8) S = 4;
        const int bn = g_force_token_tile == 128 ? 128 : (g_force_token_tile == 32 ? 32 : 64);
        if (S > 1) return GemmPlan{false, bn, 1, S};
    }
    if (g_force_token_tile > 0 || g_force_split_k > 0) {        // diagnostics: single-CTA kernel as told
        const int bn = pick_token_tile(T);
        return GemmPlan{false, bn, pick_split_k(T, N, K, bn), 0};
    }
    const double mm = sparse ? 1.0 : 1.3;                       // dense K-loop relative to sparse
    double best_t = 1e300;
    auto consider = [&](const GemmPlan& g, double t) { if (t < best_t) { best_t = t; best = g; } };
    // split-K inside clusters of 2, 3 or 4 CTAs: the K-loop shrinks and the reduction stays on chip.
    // Fitted to a sweep in a decode loop (weights from HBM, launches back to back), in us:
    //   a(bn) + q * (0.22 sparse | 0.27 dense per 128 columns) * (1 .. 1.6: co-resident CTAs share the
    //   one tensor pipe) + tokens of a tile * (scatter + finish / S).
    // All CTAs must be resident at once (tiles up to 64 tokens fit two per SM): a second wave costs
    // a whole kernel lifetime.  Clusters of 3 matter for matrices with 75..90 row tiles, where 2
    // leaves SMs with two CTAs' long K slices and 4 does not fit; they need some slack in the slot
    // count (288 CTAs in clusters of 3 did not all become resident on 296 slots).
    auto consider_cluster = [&](int bn) {
        const long tiles = static_cast<long>(rows) * ((T + bn - 1) / bn);
        const long slots = bn <= 64 ? 2L * kNumSMs : kNumSMs;
        const double a = bn == 32 ? 3.0 : (bn == 64 ? 3.3 : 3.7);
        const int tt = std::min(bn, T);
        for (int S = 2; S <= 4; ++S) {
            if (S > kb || tiles * S > slots) break;
            if (S == 3 && tiles * S * 100 > slots * 93) continue;
            const int q = (kb + S - 1) / S;
            const double per_tok = (bn == 128 ? 0.018 : 0.013) + 0.042 / S;
            const long ctas = tiles * S;
            const long per_sm = (ctas + kNumSMs - 1) / kNumSMs;
            // share of the SMs that hold two CTAs; the slowdown saturates once ~40 % of them do
            const double crowd = per_sm > 1 ? std::min(1.0, 2.5 * static_cast<double>(ctas - kNumSMs) / kNumSMs) : 0.0;
            consider(GemmPlan{false, bn, 1, S}, a + q * (sparse ? 0.22 : 0.27) * (1.0 + 0.6 * crowd) + per_tok * tt +
                                                    (per_sm > 1 ? 0.3 : 0.0) + (S == 3 ? 0.4 + 0.03 * tt : 0.0));   // 3: owner by select, not by mask
        }
    };
    if (g_allow_cluster) consider_cluster(32);
    const int bns[3] = {64, 128, 256};
    for (int bn : bns) {
        if (bn > 64 && T <= bn / 2) continue;                   // a tile mostly beyond T
        const long tiles = static_cast<long>(rows) * ((T + bn - 1) / bn);
        const double c = (bn == 256 ? 0.49 : (bn == 128 ? 0.27 : 0.23)) * mm;   // per 128 columns and wave
        const double F = 3.0 + 0.02 * bn;
        const long waves = (tiles + kNumSMs - 1) / kNumSMs;
        consider(GemmPlan{false, bn, 1, 0}, F + waves * kb * c);
        if (bn <= 128 && g_allow_cluster) consider_cluster(bn);
        if (bn == 64 && tiles * 2 <= kNumSMs) {
            // smallest split that gives at least ~100 units of work
            int sp = static_cast<int>((100 + tiles - 1) / tiles);
            if (sp > kb) sp = kb;
            while (sp > 1 && kb % sp != 0) ++sp;                // next divisor upwards (kb divides itself)
            if (sp > 1 && sp <= kb && sp <= 10) {               // many slices: the atomics dominate (33 us measured at 43)
                const double atomics = 8e-6 * static_cast<double>(T) * N * sp;
                consider(GemmPlan{false, bn, sp, 0}, F + (kb / sp) * c + 1.0 + atomics);
            }
        }
    }
    {
        const int bn = pick_pair_bn(sparse, T, N, K);
        const long tiles = static_cast<long>((N + 511) / 512) * ((T + bn - 1) / bn);
        const long waves = (tiles + kNumSMs / 2 - 1) / (kNumSMs / 2);
        consider(GemmPlan{true, bn, 1, 0}, 4.3 + 0.02 * bn + waves * kb * 0.31 * (sparse ? 1.0 : 1.65) + waves * 2.5);
    }
    {
        // One M-tile per CTA: 256-feature tiles with double-buffered accumulators.  A tile costs the same
        // whatever its token width (the MMAs' pace does not depend on it), so: fewest waves over the 74
        // pairs, then least token padding, then the widest tile.  Per 128 columns 0.205 us (sparse) /
        // 0.29 us (dense) against 0.31 / 0.43 for twice the features with two M-tiles, and no exposed
        // drain: wins for short K and for the dense kernel, loses for the sparse one at K >= 4096.
        const int cap = sparse ? kPairMaxBnSparse : kPairMaxBnDense;
        const long rows1 = (N + 255) / 256;
        int best_bn = 0;
        long best_waves = 0, best_cover = 0;
        for (int bn = cap; bn >= 128; bn -= 16) {
            const long tt = (T + bn - 1) / bn;
            const long waves = (rows1 * tt + kNumSMs / 2 - 1) / (kNumSMs / 2);
            const long cover = tt * bn;
            if (best_bn == 0 || waves < best_waves || (waves == best_waves && cover < best_cover)) {
                best_bn = bn; best_waves = waves; best_cover = cover;
            }
        }
        GemmPlan g{true, best_bn, 1, 0};
        g.mt = 1;
        consider(g, 4.3 + 0.02 * best_bn + best_waves * kb * (sparse ? 0.205 : 0.29));
    }
    return best;
}

static sbn_status run_gemm_pair(bool sparse, const int8_t* xq, const float* a_scale, int T,
                                const int8_t* wvals, const uint8_t* meta, const float* w_scale,
                                int N, int K, const float* bias, void* y, sbn_out_dtype dt,
                                int32_t* acc_out, int bn, int mt, cudaStream_t stream) {
    CUtensorMap ta, tb, te;
    bool ok;
    const uint64_t KBk = static_cast<uint64_t>(K) / kBK, NB = static_cast<uint64_t>(N) / kBM;
    if (sparse) {
        constexpr int kbs = PairConfig<true>::KBS;
        ok = encode_3d_1k(&ta, wvals, KBk * 8, NB, 8 * kbs, mt) && encode_3d_1k(&te, meta, KBk * 2, NB, 2 * kbs, mt) &&
             encode_3d_1k(&tb, xq, xq_tb8(T), KBk, bn / 16, kbs);
    } else {
        constexpr int kbs = PairConfig<false>::KBS;
        ok = encode_3d_1k(&ta, wvals, KBk * 16, NB, 16 * kbs, mt) && encode_3d_1k(&tb, xq, xq_tb8(T), KBk, bn / 16, kbs);
        te = ta;
    }
    if (!ok) return SBN_ERR_CUDA;
    PairParams pp;
    pp.g.T = T; pp.g.N = N; pp.g.K = K;
    pp.g.k_blocks_total = K / kBK;
    pp.g.k_splits = 1;
    pp.g.tb8 = static_cast<int>(xq_tb8(T));
    pp.g.a_scale = a_scale; pp.g.w_scale = w_scale; pp.g.bias = bias;
    pp.g.y = y; pp.g.out_bf16 = (dt == SBN_OUT_BF16);
    pp.g.acc_out = acc_out;
    pp.g.split_acc = nullptr; pp.g.split_counters = nullptr;
    pp.g.w_vals = wvals; pp.g.w_meta = sparse ? meta : nullptr; pp.g.w_tile_bytes = sparse ? 8192 : 16384;
    pp.g.test_skip_loads = g_test_break_waits;
    pp.g.probe = g_gemm_probe;
    pp.bn = bn;
    if (mt == 1) return sparse ? launch_pair<true, 1>(ta, tb, te, pp, stream) : launch_pair<false, 1>(ta, tb, te, pp, stream);
    return sparse ? launch_pair<true, 2>(ta, tb, te, pp, stream) : launch_pair<false, 2>(ta, tb, te, pp, stream);
}

template <bool SPARSE, int BN>
static sbn_status launch_splitk_cluster(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& te,
                                        const GemmParams& p, int cluster, cudaStream_t stream) {
    using Cfg = SplitConfig<SPARSE, BN>;
    auto kernel = bitlinear_gemm_splitk_cluster_kernel<SPARSE, BN>;
    if (!ensure_dynamic_smem<bitlinear_gemm_splitk_cluster_kernel<SPARSE, BN>>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
    const int tiles = (p.N / kBM) * ((p.T + BN - 1) / BN);
    const cudaError_t err = launch_kernel_cluster(kernel, dim3(tiles * cluster), dim3(kSplitThreads), Cfg::SMEM_BYTES, stream,
                                                  static_cast<unsigned>(cluster), ta, tb, te, p);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

static sbn_status run_gemm(bool sparse, const int8_t* xq, const float* a_scale, int T,
                           const int8_t* wvals, const uint8_t* meta, const float* w_scale,
                           int N, int K, const float* bias, void* y, sbn_out_dtype dt,
                           int32_t* acc_out, void* ws, size_t ws_bytes, cudaStream_t stream) {
    if (!xq || !a_scale || !wvals || !w_scale || !y || (sparse && !meta)) return SBN_ERR_NULL;
    if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (dt != SBN_OUT_F32 && dt != SBN_OUT_BF16) return SBN_ERR_UNSUPPORTED;
    if (misaligned(xq, 16) || misaligned(wvals, 16) || (sparse && misaligned(meta, 16)) ||
        misaligned(y, 16) || misaligned(a_scale, 4) || misaligned(w_scale, 4) ||
        (acc_out && misaligned(acc_out, 4)) || (bias && misaligned(bias, 4)))
        return SBN_ERR_ALIGN;

    const GemmPlan plan = plan_gemm(sparse, T, N, K);
    if (plan.pair)
        return run_gemm_pair(sparse, xq, a_scale, T, wvals, meta, w_scale, N, K, bias, y, dt, acc_out, plan.bn, plan.mt, stream);

    const int bn = plan.bn;
    const int splits = plan.splits;
    if (splits > 1) {
        // scratch is zero on entry (caller's duty before the first use) and the kernel re-zeroes it
        const size_t need = gemm_workspace_bytes(sparse, T, N, K);
        if (!ws || ws_bytes < need) return SBN_ERR_WORKSPACE;
        if (misaligned(ws, 16)) return SBN_ERR_ALIGN;
    }

    CUtensorMap ta, tb, te, ty;
    bool ok;
    const uint64_t NK = static_cast<uint64_t>(N) * K;
    if (sparse) {
        ok = encode_flat_1k(&ta, wvals, NK / 2, 8) && encode_flat_1k(&te, meta, NK / 8, 2);
    } else {
        ok = encode_flat_1k(&ta, wvals, NK, 16);
        te = ta;
    }
    ok = ok && encode_flat_1k(&tb, xq, xq_tiled_bytes(T, K), bn / 8);
    ok = ok && encode_2d_out(&ty, y, N, T, dt == SBN_OUT_BF16, 32);
    if (!ok) return SBN_ERR_CUDA;

    GemmParams p;
    p.T = T; p.N = N; p.K = K;
    p.k_blocks_total = K / kBK;
    p.k_splits = splits;
    p.tb8 = static_cast<int>(xq_tb8(T));
    p.a_scale = a_scale; p.w_scale = w_scale; p.bias = bias;
    p.y = y; p.out_bf16 = (dt == SBN_OUT_BF16);
    p.acc_out = acc_out;
    p.split_acc = splits > 1 ? static_cast<int32_t*>(ws) : nullptr;
    p.split_counters = splits > 1 ? reinterpret_cast<unsigned int*>(static_cast<char*>(ws) + split_acc_bytes(T, N)) : nullptr;
    p.w_vals = wvals; p.w_meta = sparse ? meta : nullptr; p.w_tile_bytes = sparse ? 8192 : 16384;
    p.test_skip_loads = g_test_break_waits;

    if (plan.cluster > 1) {
        p.k_splits = 1;
        if (sparse) return bn == 32 ? launch_splitk_cluster<true, 32>(ta, tb, te, p, plan.cluster, stream)
                         : bn == 64 ? launch_splitk_cluster<true, 64>(ta, tb, te, p, plan.cluster, stream)
                                    : launch_splitk_cluster<true, 128>(ta, tb, te, p, plan.cluster, stream);
        return bn == 32 ? launch_splitk_cluster<false, 32>(ta, tb, te, p, plan.cluster, stream)
             : bn == 64 ? launch_splitk_cluster<false, 64>(ta, tb, te, p, plan.cluster, stream)
                        : launch_splitk_cluster<false, 128>(ta, tb, te, p, plan.cluster, stream);
    }

    sbn_status st;
#define SBN_GEMM_CASE(S, B) st = launch_gemm_cfg<S, B>(ta, tb, te, ty, p, stream)
    if (sparse) {
        if (bn == 64) SBN_GEMM_CASE(true, 64); else if (bn == 128) SBN_GEMM_CASE(true, 128); else SBN_GEMM_CASE(true, 256);
    } else {
        if (bn == 64) SBN_GEMM_CASE(false, 64); else if (bn == 128) SBN_GEMM_CASE(false, 128); else SBN_GEMM_CASE(false, 256);
    }
#undef SBN_GEMM_CASE
    if (st != SBN_OK) return st;
    return SBN_OK;
}

// ---- backward GEMMs (bf16) -------------------------------------------------------------------------
struct BackwardWs {                    // W_eff^T [K][N] and x_q [T][K], both bf16
    size_t wt_off, xq_off, total;
};
static BackwardWs backward_ws_layout(int T, int N, int K) {
    BackwardWs w;
    auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
    w.wt_off = 0;
    w.xq_off = up(static_cast<size_t>(K) * N * 2);
    w.total = w.xq_off + up(static_cast<size_t>(T) * K * 2);
    return w;
}

// Output columns per tile: fewest waves over the 74 CTA pairs, weighted by what a tile costs (the A part of a
// stage is fixed, the B part grows with the tile's width).
static int pick_bf16_bn(int M, int Nn) {
    const long tiles_m = (M + 255) / 256;
    int best = 256;
    double best_cost = 1e300;
    for (int bn = 256; bn >= 128; bn -= 16) {
        const long tiles = tiles_m * ((Nn + bn - 1) / bn);
        const long waves = (tiles + kNumSMs / 2 - 1) / (kNumSMs / 2);
        const double cost = static_cast<double>(waves) * (256.0 + bn);
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

// D[M][Nn] = A[M][Kc] B[Nn][Kc]^T (bf16 in, fp32 accumulation), optionally times bf16(*scale).
// mn_major: A is stored [Kc][M] (row stride lda) and B [Kc][Nn] (row stride ldb): D = A^T B.
static sbn_status run_gemm_bf16(bool mn_major, const void* A, int M, uint64_t lda, const void* B, int Nn, uint64_t ldb, int Kc,
                                void* out, bool out_bf16, const float* scale, cudaStream_t stream,
                                bool signal_after_wait = false, bool wait_at_end = false) {
    Bf16GemmParams p;
    p.signal_after_wait = signal_after_wait ? 1 : 0;
    p.wait_at_end = wait_at_end ? 1 : 0;
    p.M = M; p.Nn = Nn; p.Kc = Kc;
    p.bn = g_force_token_tile < 0 ? std::min(256, std::max(64, (-g_force_token_tile) / 16 * 16)) : pick_bf16_bn(M, Nn);
    if (mn_major) p.bn = p.bn > 128 ? 256 : 128;                // whole 64-column blocks per CTA
    p.out = out; p.out_bf16 = out_bf16 ? 1 : 0;
    p.scale = scale;
    CUtensorMap ta, tb;
    bool ok;
    if (mn_major) {
        ok = encode_2d_bf16_sw128(&ta, A, static_cast<uint64_t>(M), static_cast<uint64_t>(Kc), lda, 64) &&
             encode_2d_bf16_sw128(&tb, B, static_cast<uint64_t>(Nn), static_cast<uint64_t>(Kc), ldb, 64);
    } else {
        ok = encode_2d_bf16_sw128(&ta, A, static_cast<uint64_t>(Kc), static_cast<uint64_t>(M), lda, 128) &&
             encode_2d_bf16_sw128(&tb, B, static_cast<uint64_t>(Kc), static_cast<uint64_t>(Nn), ldb, static_cast<uint32_t>(p.bn / 2));
    }
    if (!ok) return SBN_ERR_CUDA;
    const int tiles = ((M + 255) / 256) * ((Nn + p.bn - 1) / p.bn);
    const int pairs = tiles < kNumSMs / 2 ? tiles : kNumSMs / 2;
    cudaError_t err;
    if (mn_major) {
        if (!ensure_dynamic_smem<gemm_bf16_pair_kernel<true>>(kBf16SmemBytes)) return SBN_ERR_CUDA;
        err = launch_kernel(gemm_bf16_pair_kernel<true>, dim3(2 * pairs), dim3(kBf16Threads), kBf16SmemBytes, stream, ta, tb, p);
    } else {
        if (!ensure_dynamic_smem<gemm_bf16_pair_kernel<false>>(kBf16SmemBytes)) return SBN_ERR_CUDA;
        err = launch_kernel(gemm_bf16_pair_kernel<false>, dim3(2 * pairs), dim3(kBf16Threads), kBf16SmemBytes, stream, ta, tb, p);
    }
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// Built-in scratch for sbn_quantize_mask_pack_static_ws: part of the library image, so callers
// that cannot allocate still have somewhere to put the pass-1 partial sums.  In host code the
// symbol below is only a handle; its device address is looked up once per device.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[SBN_STATIC_SCRATCH_BYTES];
static_assert(sizeof(QmpWorkspace) <= SBN_STATIC_SCRATCH_BYTES, "built-in scratch too small");

constexpr int kMaxDevices = 64;
static void* g_static_scratch_addr[kMaxDevices] = {};
static std::mutex g_static_scratch_mutex;

// Device address of g_static_scratch on the current device (nullptr on failure).
static void* static_scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
        g_static_scratch_addr[dev] = ptr;
    }
    return g_static_scratch_addr[dev];
}

}  // namespace sbn

// ------------------------------------------------------------------------------------------------
// extern "C"
// ------------------------------------------------------------------------------------------------
using namespace sbn;

extern "C" {

size_t sbn_xq_bytes(int T, int K) {
    if (T <= 0 || K <= 0 || K % kBK != 0) return 0;
    return xq_tiled_bytes(T, K);
}

size_t sbn_workspace_bytes(int op, int T, int N, int K) {
    switch (op) {
        case SBN_OP_QUANTIZE_MASK_PACK: return sizeof(QmpWorkspace);       // one matrix; batches: sbn_batch_workspace_bytes
        case SBN_OP_QUANT_ACT: return 0;
        case SBN_OP_BACKWARD:
            if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0) return 0;
            return backward_ws_layout(T, N, K).total;
        case SBN_OP_SPARSE_BITLINEAR:
        case SBN_OP_BITLINEAR:
            if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0) return 0;
            return gemm_workspace_bytes(op == SBN_OP_SPARSE_BITLINEAR, T, N, K);
        default: return 0;
    }
}

static sbn_status quantize_mask_pack_any(const void* W, bool w_bf16, int N, int K, int n_keep, int m_group,
                                         int8_t* vals, uint8_t* meta, float* w_scale, int8_t* dense_q,
                                         const uint8_t* prev_meta, unsigned long long* flip_bits,
                                         void* ws, size_t ws_bytes, void* stream) {
    if (!W || !vals || !meta || !w_scale) return SBN_ERR_NULL;
    if (prev_meta && !flip_bits) return SBN_ERR_NULL;
    const bool p68 = n_keep == 6 && m_group == 8;
    if (!p68 && (n_keep != 2 || m_group != 4)) return SBN_ERR_UNSUPPORTED;
    if (p68 && dense_q) return SBN_ERR_UNSUPPORTED;           // the dense W_q does not depend on the pattern
    if (N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (p68 && K % (2 * kBK) != 0) return SBN_ERR_SHAPE;     // K' = 3K/2 must be a whole number of 128-column blocks
    if (!ws || ws_bytes < sizeof(QmpWorkspace)) return SBN_ERR_WORKSPACE;
    if (misaligned(W, 16) || misaligned(vals, 16) || misaligned(meta, 16) || misaligned(ws, 16) ||
        misaligned(w_scale, 4) || (dense_q && misaligned(dense_q, 16)) ||
        (prev_meta && misaligned(prev_meta, 16)) || (flip_bits && misaligned(flip_bits, 8)))
        return SBN_ERR_ALIGN;
    if (p68) {
        const QmpDesc d = qmp_make_desc(W, w_bf16, N, K, vals, meta, w_scale, nullptr, prev_meta, flip_bits);
        return launch_quantize_mask_pack_batch<68>(d, nullptr, 1, d.num_units, static_cast<QmpWorkspace*>(ws)->slot,
                                                   &static_cast<QmpWorkspace*>(ws)->generation, static_cast<cudaStream_t>(stream));
    }
    return launch_quantize_mask_pack(W, w_bf16, N, K, vals, meta, w_scale, dense_q, prev_meta, flip_bits,
                                     static_cast<QmpWorkspace*>(ws),
                                     static_cast<cudaStream_t>(stream));
}

sbn_status sbn_quantize_mask_pack(const float* W, int N, int K, int n_keep, int m_group,
                                  int8_t* vals, uint8_t* meta, float* w_scale, int8_t* dense_q,
                                  const uint8_t* prev_meta, unsigned long long* flip_bits,
                                  void* ws, size_t ws_bytes, void* stream) {
    return quantize_mask_pack_any(W, false, N, K, n_keep, m_group, vals, meta, w_scale, dense_q, prev_meta, flip_bits,
                                  ws, ws_bytes, stream);
}

sbn_status sbn_quantize_mask_pack_bf16(const void* W_bf16, int N, int K, int n_keep, int m_group,
                                       int8_t* vals, uint8_t* meta, float* w_scale, int8_t* dense_q,
                                       const uint8_t* prev_meta, unsigned long long* flip_bits,
                                       void* ws, size_t ws_bytes, void* stream) {
    return quantize_mask_pack_any(W_bf16, true, N, K, n_keep, m_group, vals, meta, w_scale, dense_q, prev_meta, flip_bits,
                                  ws, ws_bytes, stream);
}

// Batch workspace: [generation word, 256 B][job descriptors 1.., padded to 256 B][count x 148 slots].
static size_t batch_desc_bytes(int count) {
    return (static_cast<size_t>(count) * sizeof(QmpDesc) + 255) & ~static_cast<size_t>(255);
}
size_t sbn_batch_workspace_bytes(int count) {
    if (count <= 0) return 0;
    return 256 + batch_desc_bytes(count) + static_cast<size_t>(count) * sizeof(QmpWorkspace);
}

sbn_status sbn_quantize_mask_pack_batched(int count, const sbn_pack_job* jobs, void* ws, size_t ws_bytes,
                                          void* stream) {
    if (count <= 0) return SBN_ERR_SHAPE;
    if (!jobs) return SBN_ERR_NULL;
    if (!ws || ws_bytes < sbn_batch_workspace_bytes(count)) return SBN_ERR_WORKSPACE;
    if (misaligned(ws, 16)) return SBN_ERR_ALIGN;
    std::vector<QmpDesc> descs(static_cast<size_t>(count));
    for (int i = 0; i < count; ++i) {
        const sbn_pack_job& j = jobs[i];
        if (!j.W || !j.vals || !j.meta || !j.w_scale) return SBN_ERR_NULL;
        if (j.prev_meta && !j.flip_bits) return SBN_ERR_NULL;
        if (j.N <= 0 || j.K <= 0 || j.N % kBM != 0 || j.K % kBK != 0 || j.K > (1 << 20)) return SBN_ERR_SHAPE;
        if (misaligned(j.W, 16) || misaligned(j.vals, 16) || misaligned(j.meta, 16) || misaligned(j.w_scale, 4) ||
            (j.dense_q && misaligned(j.dense_q, 16)) || (j.prev_meta && misaligned(j.prev_meta, 16)) ||
            (j.flip_bits && misaligned(j.flip_bits, 8)))
            return SBN_ERR_ALIGN;
        if (j.gamma_hint && misaligned(j.gamma_hint, 4)) return SBN_ERR_ALIGN;
        descs[i] = qmp_make_desc(j.W, j.w_bf16 != 0, j.N, j.K, j.vals, j.meta, j.w_scale, j.dense_q, j.prev_meta, j.flip_bits,
                                 j.gamma_hint);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long* generation = static_cast<unsigned long long*>(ws);
    QmpDesc* descs_dev = reinterpret_cast<QmpDesc*>(static_cast<char*>(ws) + 256);
    QmpSlot* slots = reinterpret_cast<QmpSlot*>(static_cast<char*>(ws) + 256 + batch_desc_bytes(count));
    // One launch per kQmpMaxBatch matrices (the kernel keeps a little state per matrix on chip).  All jobs
    // but the first of a launch are read by the kernel from the workspace (the first travels as a kernel
    // argument).  They get there as arguments of small store kernels, a chunk at a time: nothing is staged
    // through host memory, so the call only enqueues and the caller's array is free as soon as it returns.
    for (int lo = 0; lo < count; lo += kQmpMaxBatch) {
        const int n_here = std::min(kQmpMaxBatch, count - lo);
        uint32_t max_units = 0;
        for (int i = 0; i < n_here; ++i) max_units = std::max(max_units, descs[static_cast<size_t>(lo + i)].num_units);
        // batches of up to kQmpInlineDescs matrices travel in the kernel's parameters: nothing to store first
        for (int at = 1; n_here > kQmpInlineDescs && at < n_here; at += kQmpDescChunk) {
            QmpDescChunk chunk;
            const int n = std::min(kQmpDescChunk, n_here - at);
            for (int i = 0; i < n; ++i) chunk.d[i] = descs[static_cast<size_t>(lo + at + i)];
            for (int i = n; i < kQmpDescChunk; ++i) chunk.d[i] = descs[0];
            const cudaError_t err = launch_kernel(qmp_store_descs_kernel, dim3(1), dim3(64), 0, s, chunk, descs_dev + (lo + at - 1), n);
            ++g_launch_count;
            if (err != cudaSuccess) return SBN_ERR_CUDA;
        }
        const sbn_status st = launch_quantize_mask_pack_stream(descs.data() + lo, descs_dev + lo, n_here, max_units,
                                                               slots + static_cast<size_t>(lo) * kQmpMaxCtas, generation, s);
        if (st != SBN_OK) return st;
    }
    return SBN_OK;
}

sbn_status sbn_quantize_mask_pack_static_ws(const float* W, int N, int K, int n_keep, int m_group,
                                            int8_t* vals, uint8_t* meta, float* w_scale,
                                            int8_t* dense_q, const uint8_t* prev_meta,
                                            unsigned long long* flip_bits, void* stream) {
    // size limits first: nothing below runs for a shape the built-in scratch cannot serve
    if (N > 0 && K > 0) {
        if (static_cast<long long>(N) * K > SBN_STATIC_MAX_ELEMS) return SBN_ERR_TOO_LARGE;
        if (sbn_workspace_bytes(SBN_OP_QUANTIZE_MASK_PACK, 0, N, K) > SBN_STATIC_SCRATCH_BYTES)
            return SBN_ERR_TOO_LARGE;
    }
    if (!W || !vals || !meta || !w_scale) return SBN_ERR_NULL;
    if (prev_meta && !flip_bits) return SBN_ERR_NULL;
    if (n_keep != 2 || m_group != 4) return SBN_ERR_UNSUPPORTED;
    if (N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (misaligned(W, 16) || misaligned(vals, 16) || misaligned(meta, 16) || misaligned(w_scale, 4) ||
        (dense_q && misaligned(dense_q, 16)) || (prev_meta && misaligned(prev_meta, 16)) ||
        (flip_bits && misaligned(flip_bits, 8)))
        return SBN_ERR_ALIGN;
    void* scratch = static_scratch_for_current_device();
    if (!scratch) return SBN_ERR_CUDA;
    // every slot that is read carries this call's nonce, so stale contents are harmless
    return launch_quantize_mask_pack(W, false, N, K, vals, meta, w_scale, dense_q, prev_meta, flip_bits,
                                     static_cast<QmpWorkspace*>(scratch),
                                     static_cast<cudaStream_t>(stream));
}

sbn_status sbn_quant_act(const void* x_bf16, int T, int K, int8_t* xq, float* a_scale, void* stream) {
    if (!x_bf16 || !xq || !a_scale) return SBN_ERR_NULL;
    if (T <= 0 || K <= 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (misaligned(x_bf16, 16) || misaligned(xq, 16) || misaligned(a_scale, 4)) return SBN_ERR_ALIGN;
    return launch_quant_act(x_bf16, T, K, xq, a_scale, static_cast<cudaStream_t>(stream));
}

sbn_status sbn_quant_act_expand68(const void* x_bf16, int T, int K, int8_t* xq, float* a_scale, void* stream) {
    if (!x_bf16 || !xq || !a_scale) return SBN_ERR_NULL;
    if (T <= 0 || K <= 0 || K % (2 * kBK) != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (misaligned(x_bf16, 16) || misaligned(xq, 16) || misaligned(a_scale, 4)) return SBN_ERR_ALIGN;
    return launch_quant_act<true>(x_bf16, T, K, xq, a_scale, static_cast<cudaStream_t>(stream));
}

sbn_status sbn_norm_quant_act_expand68(const void* x_bf16, int T, int K, const float* gain, float eps, int8_t* xq,
                                       float* a_scale, void* stream) {
    if (!x_bf16 || !xq || !a_scale) return SBN_ERR_NULL;
    if (T <= 0 || K <= 0 || K % (2 * kBK) != 0) return SBN_ERR_SHAPE;
    if (K > 16384) return SBN_ERR_UNSUPPORTED;
    if (!(eps >= 0.0f)) return SBN_ERR_SHAPE;
    if (misaligned(x_bf16, 16) || misaligned(xq, 16) || misaligned(a_scale, 4) || (gain && misaligned(gain, 16)))
        return SBN_ERR_ALIGN;
    return launch_norm_quant_act<true>(x_bf16, T, K, gain, eps, xq, a_scale, static_cast<cudaStream_t>(stream));
}

int sbn_expanded_k(int K, int n_keep, int m_group) {
    if (K <= 0) return 0;
    if (n_keep == 2 && m_group == 4) return K;
    if (n_keep == 6 && m_group == 8 && K % (2 * kBK) == 0 && K <= (1 << 20)) return K / 2 * 3;
    return 0;
}

sbn_status sbn_norm_quant_act(const void* x_bf16, int T, int K, const float* gain, float eps, int8_t* xq,
                              float* a_scale, void* stream) {
    if (!x_bf16 || !xq || !a_scale) return SBN_ERR_NULL;
    if (T <= 0 || K <= 0 || K % kBK != 0) return SBN_ERR_SHAPE;
    if (K > 16384) return SBN_ERR_UNSUPPORTED;
    if (!(eps >= 0.0f)) return SBN_ERR_SHAPE;
    if (misaligned(x_bf16, 16) || misaligned(xq, 16) || misaligned(a_scale, 4) || (gain && misaligned(gain, 16)))
        return SBN_ERR_ALIGN;
    return launch_norm_quant_act(x_bf16, T, K, gain, eps, xq, a_scale, static_cast<cudaStream_t>(stream));
}

sbn_status sbn_sparse_bitlinear(const int8_t* xq, const float* a_scale, int T, const int8_t* vals,
                                const uint8_t* meta, const float* w_scale, int N, int K,
                                const float* bias, void* y, sbn_out_dtype dt, int32_t* acc_out,
                                void* ws, size_t ws_bytes, void* stream) {
    return run_gemm(true, xq, a_scale, T, vals, meta, w_scale, N, K, bias, y, dt, acc_out, ws, ws_bytes,
                    static_cast<cudaStream_t>(stream));
}

sbn_status sbn_bitlinear(const int8_t* xq, const float* a_scale, int T, const int8_t* dense_q,
                         const float* w_scale, int N, int K, const float* bias, void* y,
                         sbn_out_dtype dt, int32_t* acc_out, void* ws, size_t ws_bytes, void* stream) {
    return run_gemm(false, xq, a_scale, T, dense_q, nullptr, w_scale, N, K, bias, y, dt, acc_out, ws,
                    ws_bytes, static_cast<cudaStream_t>(stream));
}

sbn_status sbn_layer_forward_host(const void* x_bf16_host, int T, int K, void* x_dev, int8_t* xq_dev,
                                  float* a_scale_dev, const int8_t* vals, const uint8_t* meta,
                                  const int8_t* dense_q, const float* w_scale, int N,
                                  const float* bias, void* y_dev, void* y_host, sbn_out_dtype dt,
                                  void* ws, size_t ws_bytes, void* stream) {
    if (!x_bf16_host || !x_dev || !xq_dev || !a_scale_dev || !y_dev || !y_host) return SBN_ERR_NULL;
    if (T <= 0 || K <= 0 || N <= 0) return SBN_ERR_SHAPE;
    if (!vals && !dense_q) return SBN_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t x_bytes = static_cast<size_t>(T) * K * 2;
    if (cudaMemcpyAsync(x_dev, x_bf16_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return SBN_ERR_CUDA;
    sbn_status st = sbn_quant_act(x_dev, T, K, xq_dev, a_scale_dev, stream);
    if (st != SBN_OK) return st;
    if (vals) {
        st = sbn_sparse_bitlinear(xq_dev, a_scale_dev, T, vals, meta, w_scale, N, K, bias, y_dev, dt, nullptr, ws, ws_bytes, stream);
    } else {
        st = sbn_bitlinear(xq_dev, a_scale_dev, T, dense_q, w_scale, N, K, bias, y_dev, dt, nullptr, ws, ws_bytes, stream);
    }
    if (st != SBN_OK) return st;
    const size_t y_bytes = static_cast<size_t>(T) * N * (dt == SBN_OUT_BF16 ? 2 : 4);
    if (cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SBN_ERR_CUDA;
    return SBN_OK;
}

// Cluster size for the 32-token few-token kernels: the cost model of plan_gemm restricted to that tile.
static int pick_cluster_32(bool sparse, int T, int N, int K) {
    const int kb = K / kBK, rows = N / kBM;
    if (g_force_split_k < 0) {                                  // diagnostics: cluster size as told
        int S = -g_force_split_k;
        S = S >= 4 ? 4 : (S == 3 ? 3 : 2);
        while (S > 2 && S > kb) --S;
        return S;
    }
    const long tiles = static_cast<long>(rows) * ((T + 31) / 32);
    const long slots = 2L * kNumSMs;
    int best_s = 2;
    double best_t = 1e300;
    for (int S = 2; S <= 4; ++S) {
        if (S > kb) break;
        if (tiles * S > slots && S > 2) break;
        if (S == 3 && tiles * S * 100 > slots * 93) continue;
        const int q = (kb + S - 1) / S;
        const long ctas = tiles * S;
        const double crowd = ctas > kNumSMs ? std::min(1.0, 2.5 * static_cast<double>(ctas - kNumSMs) / kNumSMs) : 0.0;
        const int tt = std::min(32, T);
        const double t = q * (sparse ? 0.22 : 0.27) * (1.0 + 0.6 * crowd) + (0.013 + 0.042 / S) * tt + (S == 3 ? 0.4 + 0.03 * tt : 0.0);
        if (t < best_t) { best_t = t; best_s = S; }
    }
    return best_s;
}

static sbn_status run_fused_act(bool sparse, const void* x_bf16, int T, const int8_t* wvals, const uint8_t* meta,
                                const float* w_scale, int N, int K, const float* bias, void* y, sbn_out_dtype dt,
                                int32_t* acc_out, float* a_scale_out, cudaStream_t stream) {
    if (!x_bf16 || !wvals || !w_scale || !y || (sparse && !meta)) return SBN_ERR_NULL;
    if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (dt != SBN_OUT_F32 && dt != SBN_OUT_BF16) return SBN_ERR_UNSUPPORTED;
    if (T > 256 || K < 2 * kBK) return SBN_ERR_UNSUPPORTED;           // the few-token regime only
    if (misaligned(x_bf16, 16) || misaligned(wvals, 16) || (sparse && misaligned(meta, 16)) || misaligned(y, 16) ||
        misaligned(w_scale, 4) || (acc_out && misaligned(acc_out, 4)) || (bias && misaligned(bias, 4)) ||
        (a_scale_out && misaligned(a_scale_out, 4)))
        return SBN_ERR_ALIGN;
    CUtensorMap ta, te;
    bool ok;
    const uint64_t NK = static_cast<uint64_t>(N) * K;
    if (sparse) {
        ok = encode_flat_1k(&ta, wvals, NK / 2, 8) && encode_flat_1k(&te, meta, NK / 8, 2);
    } else {
        ok = encode_flat_1k(&ta, wvals, NK, 16);
        te = ta;
    }
    if (!ok) return SBN_ERR_CUDA;
    FusedActParams fp;
    GemmParams& p = fp.g;
    p.T = T; p.N = N; p.K = K;
    p.k_blocks_total = K / kBK;
    p.k_splits = 1;
    p.tb8 = 0;
    p.a_scale = nullptr; p.w_scale = w_scale; p.bias = bias;
    p.y = y; p.out_bf16 = (dt == SBN_OUT_BF16);
    p.acc_out = acc_out;
    p.split_acc = nullptr; p.split_counters = nullptr;
    p.w_vals = wvals; p.w_meta = sparse ? meta : nullptr; p.w_tile_bytes = sparse ? 8192 : 16384;
    fp.x_bf16 = x_bf16;
    fp.a_scale_out = a_scale_out;
    const int tiles = (N / kBM) * ((T + 31) / 32);
    const int cluster = pick_cluster_32(sparse, T, N, K);
    cudaError_t err;
    if (sparse) {
        using Cfg = FusedActConfig<true>;
        if (!ensure_dynamic_smem<bitlinear_gemm_fused_act_cluster_kernel<true>>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
        err = launch_kernel_cluster(bitlinear_gemm_fused_act_cluster_kernel<true>, dim3(tiles * cluster), dim3(kSplitThreads),
                                    Cfg::SMEM_BYTES, stream, static_cast<unsigned>(cluster), ta, te, fp);
    } else {
        using Cfg = FusedActConfig<false>;
        if (!ensure_dynamic_smem<bitlinear_gemm_fused_act_cluster_kernel<false>>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
        err = launch_kernel_cluster(bitlinear_gemm_fused_act_cluster_kernel<false>, dim3(tiles * cluster), dim3(kSplitThreads),
                                    Cfg::SMEM_BYTES, stream, static_cast<unsigned>(cluster), ta, te, fp);
    }
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

sbn_status sbn_quant_act_sparse_bitlinear(const void* x_bf16, int T, const int8_t* vals, const uint8_t* meta,
                                          const float* w_scale, int N, int K, const float* bias, void* y,
                                          sbn_out_dtype dt, int32_t* acc_out, float* a_scale_out, void* stream) {
    return run_fused_act(true, x_bf16, T, vals, meta, w_scale, N, K, bias, y, dt, acc_out, a_scale_out,
                         static_cast<cudaStream_t>(stream));
}

sbn_status sbn_quant_act_bitlinear(const void* x_bf16, int T, const int8_t* dense_q, const float* w_scale, int N, int K,
                                   const float* bias, void* y, sbn_out_dtype dt, int32_t* acc_out, float* a_scale_out,
                                   void* stream) {
    return run_fused_act(false, x_bf16, T, dense_q, nullptr, w_scale, N, K, bias, y, dt, acc_out, a_scale_out,
                         static_cast<cudaStream_t>(stream));
}

sbn_status sbn_pack_vals2(const int8_t* vals, int N, int K, uint8_t* vals2, void* stream) {
    if (!vals || !vals2) return SBN_ERR_NULL;
    if (N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (misaligned(vals, 16) || misaligned(vals2, 16)) return SBN_ERR_ALIGN;
    return launch_pack_vals2(vals, N, K, vals2, static_cast<cudaStream_t>(stream));
}

sbn_status sbn_sparse_bitlinear_packed(const int8_t* xq, const float* a_scale, int T, const uint8_t* vals2,
                                       const uint8_t* meta, const float* w_scale, int N, int K, const float* bias,
                                       void* y, sbn_out_dtype dt, int32_t* acc_out, void* stream) {
    if (!xq || !a_scale || !vals2 || !meta || !w_scale || !y) return SBN_ERR_NULL;
    if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (dt != SBN_OUT_F32 && dt != SBN_OUT_BF16) return SBN_ERR_UNSUPPORTED;
    if (T > 1024 || K < 2 * kBK) return SBN_ERR_UNSUPPORTED;          // the few-token regime only
    if (misaligned(xq, 16) || misaligned(vals2, 16) || misaligned(meta, 16) || misaligned(y, 16) || misaligned(a_scale, 4) ||
        misaligned(w_scale, 4) || (acc_out && misaligned(acc_out, 4)) || (bias && misaligned(bias, 4)))
        return SBN_ERR_ALIGN;
    using Cfg = PackedSplitConfig;
    CUtensorMap tb;
    if (!encode_flat_1k(&tb, xq, xq_tiled_bytes(T, K), Cfg::BN / 8)) return SBN_ERR_CUDA;
    GemmParams p;
    p.T = T; p.N = N; p.K = K;
    p.k_blocks_total = K / kBK;
    p.k_splits = 1;
    p.tb8 = static_cast<int>(xq_tb8(T));
    p.a_scale = a_scale; p.w_scale = w_scale; p.bias = bias;
    p.y = y; p.out_bf16 = (dt == SBN_OUT_BF16);
    p.acc_out = acc_out;
    p.split_acc = nullptr; p.split_counters = nullptr;
    p.w_vals = vals2; p.w_meta = meta; p.w_tile_bytes = kVals2TileBytes;
    const int tiles = (N / kBM) * ((T + Cfg::BN - 1) / Cfg::BN);
    const int cluster = pick_cluster_32(true, T, N, K);
    if (!ensure_dynamic_smem<bitlinear_gemm_packed_cluster_kernel>(Cfg::SMEM_BYTES)) return SBN_ERR_CUDA;
    const cudaError_t err = launch_kernel_cluster(bitlinear_gemm_packed_cluster_kernel, dim3(tiles * cluster), dim3(kSplitThreads),
                                                  Cfg::SMEM_BYTES, static_cast<cudaStream_t>(stream), static_cast<unsigned>(cluster), tb, p);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

static sbn_status canonical_any(bool to_tiled, const void* vals_in, const void* meta_in, int N, int K, void* vals_out,
                                void* meta_out, void* stream) {
    if ((!vals_in) != (!vals_out) || (!meta_in) != (!meta_out) || (!vals_in && !meta_in)) return SBN_ERR_NULL;
    if (N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    if (misaligned(vals_in, 16) || misaligned(vals_out, 16) || misaligned(meta_in, 16) || misaligned(meta_out, 16))
        return SBN_ERR_ALIGN;
    if ((vals_in && vals_in == vals_out) || (meta_in && meta_in == meta_out)) return SBN_ERR_UNSUPPORTED;   // not in place
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return to_tiled ? launch_canonical_layout<true>(vals_in, vals_out, meta_in, meta_out, N, K, s)
                    : launch_canonical_layout<false>(vals_in, vals_out, meta_in, meta_out, N, K, s);
}

sbn_status sbn_unpack_canonical(const int8_t* vals, const uint8_t* meta, int N, int K, int8_t* vals_out,
                                uint8_t* meta_out, void* stream) {
    return canonical_any(false, vals, meta, N, K, vals_out, meta_out, stream);
}

sbn_status sbn_tile_canonical(const int8_t* vals_plain, const uint8_t* meta_plain, int N, int K, int8_t* vals,
                              uint8_t* meta, void* stream) {
    return canonical_any(true, vals_plain, meta_plain, N, K, vals, meta, stream);
}

sbn_status sbn_bitlinear_backward(const void* dY_bf16, int T, const int8_t* xq, const float* a_scale, const int8_t* vals,
                                  const uint8_t* meta, const float* w_scale, int N, int K, void* dX_bf16, float* dW,
                                  void* ws, size_t ws_bytes, void* stream) {
    if (!dY_bf16 || (!dX_bf16 && !dW)) return SBN_ERR_NULL;
    if (dX_bf16 && (!vals || !meta || !w_scale)) return SBN_ERR_NULL;
    if (dW && (!xq || !a_scale)) return SBN_ERR_NULL;
    if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0 || K > (1 << 20)) return SBN_ERR_SHAPE;
    const BackwardWs lay = backward_ws_layout(T, N, K);
    if (!ws || ws_bytes < lay.total) return SBN_ERR_WORKSPACE;
    if (misaligned(dY_bf16, 16) || misaligned(ws, 256) || (dX_bf16 && (misaligned(dX_bf16, 16) || misaligned(vals, 16) || misaligned(meta, 16) || misaligned(w_scale, 4))) ||
        (dW && (misaligned(dW, 16) || misaligned(xq, 16) || misaligned(a_scale, 4))))
        return SBN_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);
    uint16_t* Wt = reinterpret_cast<uint16_t*>(base + lay.wt_off);
    uint16_t* XT = reinterpret_cast<uint16_t*>(base + lay.xq_off);
    const int KB = K / kBK, NB = N / kBM;
    // Operands first (two small memory-bound kernels), then the GEMMs.  With both gradients wanted the
    // weight-gradient GEMM goes first and the input-gradient GEMM moves into the pairs its last wave
    // leaves idle (Bf16GemmParams: signal_after_wait / wait_at_end): the two do not depend on each other.
    const bool both = dX_bf16 != nullptr && dW != nullptr;
    if (dX_bf16) {
        if (launch_kernel(weff_t_bf16_kernel, dim3(KB * NB), dim3(kPrepThreads), 0, s, reinterpret_cast<const uint8_t*>(vals), meta, N, K, Wt) != cudaSuccess)
            return SBN_ERR_CUDA;
        ++g_launch_count;
    }
    if (dW) {
        const unsigned blocks = static_cast<unsigned>(std::min<size_t>((static_cast<size_t>(T) * (K / 16) + kPrepThreads - 1) / kPrepThreads,
                                                                           static_cast<size_t>(device_sm_count()) * 8));
        if (launch_kernel(xq_bf16_kernel, dim3(blocks), dim3(kPrepThreads), 0, s, reinterpret_cast<const uint8_t*>(xq), a_scale, T, K, XT) != cudaSuccess)
            return SBN_ERR_CUDA;
        ++g_launch_count;
        // dW[n][k] = sum_t dY[t][n] x_q[t][k]
        // both operands as they lie in memory, token-major: dY [T][N] and x_q [T][K] (bf16 copy of the
        // fake-quantised activations); the MMA reads them MN-major, the contraction runs down the rows
        const sbn_status st = run_gemm_bf16(true, dY_bf16, N, static_cast<uint64_t>(N), XT, K, static_cast<uint64_t>(K), T, dW, false, nullptr, s,
                                            both, false);
        if (st != SBN_OK) return st;
    }
    if (dX_bf16) {
        // dX[t][k] = bf16(scale) * sum_n dY[t][n] W_eff[n][k]: A = dY [T][N], B = W_eff^T [K][N]
        const sbn_status st = run_gemm_bf16(false, dY_bf16, T, static_cast<uint64_t>(N), Wt, K, static_cast<uint64_t>(N), N, dX_bf16, true, w_scale, s,
                                            false, both);
        if (st != SBN_OK) return st;
    }
    return SBN_OK;
}

sbn_status sbn_check_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SBN_ERR_CUDA;
    int h = 0;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return SBN_ERR_CUDA;
    if (h != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
        return static_cast<sbn_status>(h);
    }
    return SBN_OK;
}

const char* sbn_status_string(sbn_status s) {
    switch (s) {
        case SBN_OK: return "ok";
        case SBN_ERR_NULL: return "a required pointer is NULL";
        case SBN_ERR_SHAPE: return "bad shape (need T >= 1, N % 128 == 0, K % 128 == 0)";
        case SBN_ERR_ALIGN: return "pointer not 16-byte aligned";
        case SBN_ERR_UNSUPPORTED: return "unsupported pattern, dtype or op";
        case SBN_ERR_WORKSPACE: return "workspace missing or too small";
        case SBN_ERR_CUDA: return "CUDA call failed";
        case SBN_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case SBN_ERR_TOO_LARGE: return "problem larger than the library's built-in scratch can serve";
        default: return "unknown status";
    }
}

void sbn_plan_gemm(int sparse, int T, int N, int K, int* out4) {
    if (!out4) return;
    out4[0] = out4[1] = out4[2] = out4[3] = 0;
    if (T <= 0 || N <= 0 || K <= 0 || N % kBM != 0 || K % kBK != 0) return;
    const GemmPlan g = plan_gemm(sparse != 0, T, N, K);
    out4[0] = g.pair ? (g.mt == 1 ? 3 : 2) : (g.cluster > 1 ? 1 : 0);
    out4[1] = g.bn;
    out4[2] = g.splits;
    out4[3] = g.cluster;
}

sbn_status sbn_set_wait_test(int break_waits, unsigned long long wait_limit_us) {
    const unsigned long long ns = wait_limit_us == 0ull ? kWaitLimitNs : wait_limit_us * 1000ull;
    if (cudaMemcpyToSymbol(g_wait_limit_ns, &ns, sizeof(ns)) != cudaSuccess) return SBN_ERR_CUDA;
    g_test_break_waits = break_waits ? 1 : 0;
    return SBN_OK;
}

void sbn_set_gemm_probe(int flags) { g_gemm_probe = flags; }

void sbn_set_gemm_tuning(int token_tile, int split_k) {
    g_force_token_tile = token_tile;
    g_force_split_k = split_k;
}

unsigned long long sbn_launch_count(void) { return g_launch_count.load(); }

}  // extern "C"
