// Part 1 of the path: absmean ternary quantisation (Eq. 1), 2:4 magnitude mask from the master
// weights (Eq. 2), W_eff = W_q (.) M (Eq. 3), compressed value + metadata layout.
//
// gamma needs the whole matrix before any element can be rounded, but almost every element can be
// rounded correctly from an ESTIMATE of gamma: W_q = sign(w) [ |w| >= thr(gamma) ] and only the
// few |w| that lie within a few percent of thr depend on its exact value.  One persistent kernel
// (one 1024-thread CTA per SM) therefore reads W ONCE, for one matrix or a batch of them.  This file
// holds the building blocks and the phase-by-phase kernel that the 6:8 pattern uses; the 2:4 pattern
// runs the same phases as one uninterrupted stream (quantize_mask_pack_stream.cuh).  The phases:
//
//   sample   every CTA adds |w| over the same 256 scattered 512 B units of the matrix (128 KB,
//            L2-served for all CTAs but the first; 64 units for matrices below 33 M weights)
//            -> gamma_est, and brackets the threshold: thr_lo ~ thr(0.97 gamma_est),
//            thr_hi ~ thr(1.03 gamma_est) (0.96 / 1.04 with the small sample);
//   pass 1   every CTA owns a contiguous range of (row, 128-column) units and streams it:
//            sum|W| in fp64 (the exact gamma), top 2 of 4 per group (Eq. 2: the mask does not
//            depend on gamma), metadata, flip count, and the two kept values ternarised
//            PROVISIONALLY: |w| >= thr_hi -> +-1 and |w| < thr_lo -> 0 are final whatever gamma
//            turns out to be inside the bracket; the others (~2 % for Gaussian weights) are
//            appended as {byte position, w} to a list in shared memory;
//   exchange every CTA publishes {tag, partial sum} in the workspace and waits (bounded) until all
//            slots carry this execution's tag -- no atomics, nothing to initialise; every CTA then
//            adds the 148 partials in the same fixed order, so all get the same bits, run after
//            run.  The tag joins the host's per-call nonce with a generation word that lives in
//            the workspace and that CTA 0 advances at the end of every execution: stale slots of
//            earlier calls never match, and neither do those of an earlier REPLAY of the same
//            captured launch (whose nonce is frozen in the graph);
//   fix-up   with the exact thr: if thr_lo <= thr <= thr_hi (and the list did not overflow) only
//            the listed bytes are rewritten -- the result is exactly Eq. 1, not an approximation.
//            Otherwise (a sample that misrepresents the matrix, the 1e-5 clamp, a request for the
//            dense W_q, which needs all four weights of a group) the CTA reads its range again
//            and ternarises everything with the exact thr: slower, same result.
//
// HBM traffic per parameter: 4 B read + 0.625 B written.  16 B loads per lane, a warp covers one
// 512 B unit; a warp store covers whole 64 B (vals), 128 B (dense W_q) or 16 B (metadata) rows of
// an operand tile (tiled layouts, see layouts.cuh).
//
// Ternarisation without a per-element division: W_q = sign(w) * [ fl(|w| / scale) > 0.5 ]
// (round-half-even sends exactly 0.5 to 0, everything above to >= 1, the clamp caps at 1).
// Correctly rounded division is monotone in |w|, so there is one fp32 threshold thr with
// fl(a / scale) > 0.5  <=>  a >= thr.  thr is found once per matrix with real IEEE divisions
// and the per-element work is a compare.
#pragma once

#include <algorithm>

#include "sbn_common.cuh"
#include "layouts.cuh"

namespace sbn {

constexpr int kQmpThreads = 1024;
constexpr int kQmpWarps = kQmpThreads / 32;
constexpr int kQmpMaxCtas = kNumSMs;                       // one CTA per SM, all co-resident
constexpr int kQmpListCap = 8192;                          // undecided entries per CTA and matrix
constexpr int kQmpSmemBytes = 2 * kQmpListCap * 8;         // two lists (consecutive matrices of a batch)
constexpr int kQmpSampleUnits = 256;                       // units in the gamma_est sample of a large matrix
constexpr float kQmpBracket = 0.03f;                       // gamma_est * (1 -+ this) brackets gamma
// Matrices below 2^18 units (33.5 M weights) are sampled at a quarter of that with a wider bracket:
// there the sample is a visible part of the kernel's time (2.5 us of ~25), and 8192 weights still put
// the bracket at 4.8 standard errors of the mean for Gaussian weights.  Large matrices keep the
// larger sample, which also holds for heavy-tailed weights.
constexpr int kQmpSampleUnitsSmall = 64;
constexpr float kQmpBracketSmall = 0.04f;
constexpr uint32_t kQmpSmallMatrixUnits = 1u << 18;
__host__ __device__ inline uint32_t qmp_sample_units(uint32_t num_units) {
    const uint32_t want = num_units < kQmpSmallMatrixUnits ? kQmpSampleUnitsSmall : kQmpSampleUnits;
    return num_units < want ? num_units : want;
}

struct QmpSlot {                 // one per CTA, 16 B
    unsigned long long nonce;    // tag of the execution that wrote `partial`
    double partial;              // this CTA's sum |W|
};
// What a single-matrix call leaves behind for the next call on the same workspace: the scale it found,
// tagged with the matrix it belongs to.  The next call on the same matrix (a training loop re-packs the
// same buffers every step) takes it as its estimate of gamma -- no sample, a narrow bracket -- exactly as
// if the caller had passed it as a hint; anything else in these bytes (an uninitialised workspace, another
// matrix) fails the tag and is ignored.
struct __align__(16) QmpMemo {
    unsigned long long magic;
    const void* W;
    uint32_t num_units;
    float scale;
};
constexpr unsigned long long kQmpMemoMagic = 0x71A93C5E2D84B6F1ull;
struct QmpWorkspace {            // layout of the caller's workspace
    QmpSlot slot[kQmpMaxCtas];
    unsigned long long generation;   // advanced by one per execution on this workspace (any start value)
    unsigned long long pad_;
    QmpMemo memo;
    unsigned long long pad2_;
};
// Tag of one execution: the call's nonce (low word, never 0) under the workspace's generation.
__device__ __forceinline__ unsigned long long qmp_tag(unsigned long long nonce, unsigned long long generation) {
    return (generation << 32) | (nonce & 0xFFFFFFFFull);
}

__device__ __forceinline__ unsigned long long global_timer_ns_qmp() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Smallest fp32 a with fl(a / scale) > 0.5, searched around 0.5 * scale with IEEE divisions.
__device__ __forceinline__ float ternary_threshold(float scale) {
    float a = 0.5f * scale;
    for (int it = 0; it < 8 && __fdiv_rn(a, scale) > 0.5f; ++it) a = __uint_as_float(__float_as_uint(a) - 1u);
    for (int it = 0; it < 16 && !(__fdiv_rn(a, scale) > 0.5f); ++it) a = __uint_as_float(__float_as_uint(a) + 1u);
    return a;
}

// Eq. 2 for one group: the two largest |w| of four (ranking on the fp32 master weights; on equal
// magnitudes the lower column wins).  Returns the nibble i0 | i1 << 2 (i0 < i1) and the two kept
// weights in column order.  The winners of the pairs (0,1) and (2,3) are the answer unless the
// loser of one pair still beats the winner of the other:
//   min(a0,a1) >= max(a2,a3)  ->  columns 0,1   (a tie goes to the lower column, hence >=)
//   min(a2,a3) >  max(a0,a1)  ->  columns 2,3   (and hence > here)
__device__ __forceinline__ uint32_t select_pair(const float4 w, float& v0, float& v1) {
    const float a0 = fabsf(w.x), a1 = fabsf(w.y), a2 = fabsf(w.z), a3 = fabsf(w.w);
    const bool c01 = a0 >= a1, c23 = a2 >= a3;
    const bool both01 = fminf(a0, a1) >= fmaxf(a2, a3);
    const bool both23 = fminf(a2, a3) > fmaxf(a0, a1);
    v0 = c01 ? w.x : w.y;
    v1 = c23 ? w.z : w.w;
    uint32_t nib = (c01 ? 0u : 1u) | (c23 ? 8u : 12u);
    if (both01) { v0 = w.x; v1 = w.y; nib = 4u; }
    if (both23) { v0 = w.z; v1 = w.w; nib = 14u; }
    return nib;
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Eq. 1 for four elements as four bytes (+1 -> 0x01, -1 -> 0xFF, 0 -> 0x00; thr: see the header),
// lowest byte = first argument.  The sign bytes come from byte permutes in sign-replication mode.
__device__ __forceinline__ uint32_t ternary_bytes4(float w0, float w1, float w2, float w3, float thr) {
    const uint32_t s01 = prmt(__float_as_uint(w0), __float_as_uint(w1), 0x00FBu);   // bytes 0,1: 0xFF if negative
    const uint32_t s23 = prmt(__float_as_uint(w2), __float_as_uint(w3), 0x00FBu);
    const uint32_t sgn = prmt(s01, s23, 0x5410u);
    const uint32_t keep = (fabsf(w0) >= thr ? 0x000000FFu : 0u) | (fabsf(w1) >= thr ? 0x0000FF00u : 0u) |
                          (fabsf(w2) >= thr ? 0x00FF0000u : 0u) | (fabsf(w3) >= thr ? 0xFF000000u : 0u);
    return (sgn | 0x01010101u) & keep;
}
__device__ __forceinline__ uint32_t ternary_bytes2(float w0, float w1, float thr) {
    const uint32_t sgn = prmt(__float_as_uint(w0), __float_as_uint(w1), 0x00FBu);
    const uint32_t keep = (fabsf(w0) >= thr ? 0x00FFu : 0u) | (fabsf(w1) >= thr ? 0xFF00u : 0u);
    return (sgn | 0x0101u) & keep;
}

__device__ __forceinline__ uint32_t nibble_to_mask(uint32_t nib) {
    return (1u << (nib & 3u)) | (1u << ((nib >> 2) & 3u));
}

constexpr int kQmpPrefetchAhead = 3;                       // pass 1 iterations (128 units = 64 KB each) ahead

// Sum of `v` over the CTA in a fixed order; identical in every thread.
__device__ __forceinline__ double qmp_block_sum(double v, double* s_warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) s_warp[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kQmpWarps; ++w) t += s_warp[w];
    __syncthreads();
    return t;
}

__device__ __forceinline__ double abs_sum4(const float4 v) {
    return ((double)fabsf(v.x) + (double)fabsf(v.y)) + ((double)fabsf(v.z) + (double)fabsf(v.w));
}

// One matrix of a batch (device-visible copy of the call's arguments).
struct QmpDesc {
    const void* W;                     // fp32 [N][K], or bf16 [N][K] when w_bf16
    uint16_t* vals;
    uint8_t* meta;
    float* w_scale;
    uint32_t* dense_q;                 // or null
    const uint8_t* prev_meta;          // or null
    unsigned long long* flip_bits;     // or null
    const float* gamma_hint;           // or null: the caller's estimate of gamma (e.g. the previous step's scale)
    uint32_t num_units;                // N * K / 128
    uint32_t KB;                       // K / 128
    uint32_t w_bf16;                   // master weights are bf16 (Sec. 2.2 keeps them "e.g. in bf16")
};

struct QmpRange {                      // this CTA's share of one matrix
    uint32_t u_begin, u_end;
};
struct QmpEntry {                      // one undecided kept value
    uint32_t byte_off;                 // its byte in vals
    float w;
};

// One group (4 consecutive weights) of unit u for lane `lane` (a warp covers the unit's 32 groups).
template <bool BF16>
__device__ __forceinline__ float4 qmp_load_group(const void* W, size_t u, int lane) {
    if constexpr (BF16) {
        const uint2 v = __ldg(static_cast<const uint2*>(W) + u * 32 + lane);
        return make_float4(bf16lo_to_f32(v.x), bf16hi_to_f32(v.x), bf16lo_to_f32(v.y), bf16hi_to_f32(v.y));
    } else {
        return __ldg(static_cast<const float4*>(W) + u * 32 + lane);
    }
}
// Two adjacent groups of unit u for lane l16 of a half-warp (16 lanes cover the unit).
template <bool BF16>
__device__ __forceinline__ void qmp_load_group_pair(const void* W, size_t u, uint32_t l16, float4& a, float4& b) {
    if constexpr (BF16) {
        const uint4 v = __ldg(static_cast<const uint4*>(W) + u * 16 + l16);
        a = make_float4(bf16lo_to_f32(v.x), bf16hi_to_f32(v.x), bf16lo_to_f32(v.y), bf16hi_to_f32(v.y));
        b = make_float4(bf16lo_to_f32(v.z), bf16hi_to_f32(v.z), bf16lo_to_f32(v.w), bf16hi_to_f32(v.w));
    } else {
        const float4* src = static_cast<const float4*>(W) + u * 32 + 2 * l16;
        a = __ldg(src);
        b = __ldg(src + 1);
    }
}

__device__ __forceinline__ QmpRange qmp_range(const QmpDesc& d) {
    QmpRange r;
    const uint32_t per = (d.num_units + gridDim.x - 1) / gridDim.x;
    r.u_begin = min(d.num_units, blockIdx.x * per);
    r.u_end = min(d.num_units, r.u_begin + per);
    return r;
}

// gamma_est: mean |w| over kQmpSampleUnits units scattered over the matrix (the same units in every
// CTA; a multiplicative hash keeps them off any row / column-block period).  fp32 is plenty here.
template <bool BF16>
__device__ __forceinline__ float qmp_sample_gamma(const QmpDesc& d, double* s_warp) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t n_s = qmp_sample_units(d.num_units);
    const uint32_t stride = d.num_units / n_s;                        // >= 1
    float acc = 0.0f;
    constexpr int kPerWarp = kQmpSampleUnits / kQmpWarps;
    float4 v[kPerWarp];
#pragma unroll
    for (int i = 0; i < kPerWarp; ++i) {                  // all loads of the warp in flight at once
        const uint32_t sidx = warp + i * kQmpWarps;
        const uint32_t u = sidx * stride + ((sidx * 2654435761u) >> 8) % stride;
        v[i] = sidx < n_s ? qmp_load_group<BF16>(d.W, u, lane) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < kPerWarp; ++i) acc += (fabsf(v[i].x) + fabsf(v[i].y)) + (fabsf(v[i].z) + fabsf(v[i].w));
    const double total = qmp_block_sum(static_cast<double>(acc), s_warp);
    return static_cast<float>(total / (static_cast<double>(n_s) * 128.0));
}

// Appends the undecided ones of four consecutive kept values (bytes byte_off .. byte_off + 3 of vals).
template <int CAP = kQmpListCap>
__device__ __forceinline__ void qmp_list_undecided(const float (&k)[4], const float thr_lo, const float thr_hi,
                                                   const uint32_t byte_off, QmpEntry* list, unsigned int* list_count) {
    bool und[4];
    unsigned int cnt = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float a = fabsf(k[i]);
        und[i] = a >= thr_lo && a < thr_hi;
        cnt += und[i] ? 1u : 0u;
    }
    if (cnt != 0u) {                                       // a few percent of the lanes get here
        unsigned int at = atomicAdd(list_count, cnt);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (und[i]) {
                if (at < static_cast<unsigned int>(CAP)) { list[at].byte_off = byte_off + i; list[at].w = k[i]; }
                ++at;
            }
        }
    }
}

// Ternarise a whole range again with the exact threshold (the path taken when the bracket missed,
// the list overflowed or the dense W_q is wanted): a warp per unit, four units at a time, newest
// first (what pass 1 read last is still in L2).
template <bool BF16>
__device__ __forceinline__ void qmp_pass2_full(const QmpDesc& d, const QmpRange rg, float thr) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t KB = d.KB;
    const uint32_t n_units = rg.u_end - rg.u_begin;
    const bool write_dense = d.dense_q != nullptr;
    const int step_n = static_cast<int>(kQmpWarps / KB), step_kb = static_cast<int>(kQmpWarps % KB);
    int n_cur = 0, kb_cur = 0;
    if (static_cast<uint32_t>(warp) < n_units) {
        const uint32_t u_first = rg.u_begin + (n_units - 1 - warp);
        n_cur = static_cast<int>(u_first / KB);
        kb_cur = static_cast<int>(u_first - static_cast<uint32_t>(n_cur) * KB);
    }
    for (uint32_t i0 = warp; i0 < n_units; i0 += 4 * kQmpWarps) {
        float4 w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t i = i0 + q * kQmpWarps;
            w[q] = (i < n_units) ? qmp_load_group<BF16>(d.W, rg.u_begin + (n_units - 1 - i), lane)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t i = i0 + q * kQmpWarps;
            if (i < n_units) {
                const size_t tile_idx = static_cast<size_t>(static_cast<uint32_t>(n_cur) >> 7) * KB + static_cast<uint32_t>(kb_cur);
                const uint32_t rr = static_cast<uint32_t>(n_cur) & 127u;
                n_cur -= step_n;
                kb_cur -= step_kb;
                if (kb_cur < 0) { kb_cur += static_cast<int>(KB); --n_cur; }
                float k0, k1;
                select_pair(w[q], k0, k1);
                // compressed columns 2*lane, 2*lane+1 of this 64 B tile row
                d.vals[((tile_idx << 13) + vals_in_tile(rr, 2u * lane)) >> 1] = static_cast<uint16_t>(ternary_bytes2(k0, k1, thr));
                if (write_dense)
                    d.dense_q[((tile_idx << 14) + sw128_in_tile(rr, 4u * lane)) >> 2] =
                        ternary_bytes4(w[q].x, w[q].y, w[q].z, w[q].w, thr);
            }
        }
    }
}

// The pass of the 6:8 pattern (quantize_mask_pack68.cuh; FINAL = values only, exact threshold).
template <bool BF16, bool FINAL>
__device__ __forceinline__ double qmp68_pass(const QmpDesc& d, const QmpRange rg, const float thr_lo, const float thr_hi,
                                             QmpEntry* list, unsigned int* list_count, double* s_warp,
                                             unsigned int& flips);

// Batch of `count` matrices in one persistent launch, software-pipelined over the matrices:
//   S+P1(0) | S+P1(1) F(0) | S+P1(2) F(1) | ... | F(count-1)        (S sample, F exchange + fix-up)
// so by the time a CTA needs gamma of matrix m, every CTA has long published its partial for m,
// and the per-launch and per-exchange latencies are paid once per batch, not once per matrix.
// The two undecided lists alternate between consecutive matrices.  `first` is matrix 0 (passed by
// value), `rest` matrices 1.. in global memory.  PATTERN: 68 (the 2:4 pattern has its own kernel).
template <int PATTERN>
__global__ void __launch_bounds__(kQmpThreads, 1)
quantize_mask_pack_kernel(const QmpDesc first, const QmpDesc* __restrict__ rest, int count,
                          QmpSlot* slots, unsigned long long* generation, unsigned long long call_nonce,
                          int test_withhold_slot) {
    extern __shared__ QmpEntry s_list[];                // [2][kQmpListCap]
    __shared__ double s_warp[kQmpWarps];
    __shared__ float s_thr;
    __shared__ int s_ok;
    __shared__ unsigned int s_flips[kQmpWarps];
    __shared__ unsigned long long s_flip_total[2];
    __shared__ unsigned int s_list_count[2];
    __shared__ float s_bracket[2][2];                   // [matrix parity][lo, hi]

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_ok = 1;
    __syncthreads();
    // No early signal to the next kernel of the stream: this kernel writes packed weights, and the
    // GEMM kernels fetch weights before their own dependency wait (see sbn_common.cuh).
    pdl_wait();
    // stable for the whole execution: CTA 0 advances it only after it has seen every CTA's last slot,
    // and every CTA reads it here, before it publishes anything
    const unsigned long long gen0 = *reinterpret_cast<volatile unsigned long long*>(generation);
    const unsigned long long nonce = qmp_tag(call_nonce, gen0);

    QmpDesc d_prev = first;
    QmpRange rg_prev = {0u, 0u};
    for (int m = 0; m <= count; ++m) {
        // ---- sample + pass 1 of matrix m, publish its partial
        QmpDesc d_cur = first;
        QmpRange rg_cur = {0u, 0u};
        if (m < count) {
            if (m > 0) d_cur = rest[m - 1];
            rg_cur = qmp_range(d_cur);
            const int par = m & 1;
            const float gamma_est = d_cur.w_bf16 ? qmp_sample_gamma<true>(d_cur, s_warp) : qmp_sample_gamma<false>(d_cur, s_warp);
            if (threadIdx.x == 0) {
                s_list_count[par] = 0u;
                // any lo <= hi will do (the exact threshold is checked against them later), so no
                // divisions here: thr(scale) is 0.5 * scale to within a few ulps
                const float b = d_cur.num_units < kQmpSmallMatrixUnits ? kQmpBracketSmall : kQmpBracket;
                s_bracket[par][0] = 0.5f * fmaxf(gamma_est * (1.0f - b), kEps) * (1.0f - 1e-6f);
                s_bracket[par][1] = 0.5f * fmaxf(gamma_est * (1.0f + b), kEps) * (1.0f + 1e-6f);
            }
            __syncthreads();
            unsigned int flips = 0;
            double mine;
            static_assert(PATTERN == 68, "the 2:4 pattern runs in quantize_mask_pack_stream_kernel");
            mine = d_cur.w_bf16
                ? qmp68_pass<true, false>(d_cur, rg_cur, s_bracket[par][0], s_bracket[par][1], s_list + par * kQmpListCap,
                                          &s_list_count[par], s_warp, flips)
                : qmp68_pass<false, false>(d_cur, rg_cur, s_bracket[par][0], s_bracket[par][1], s_list + par * kQmpListCap,
                                           &s_list_count[par], s_warp, flips);
            // this CTA's flip count of matrix m; it is added to the global counter one phase later,
            // after the exchange has shown that CTA 0 zeroed that counter
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) flips += __shfl_xor_sync(0xFFFFFFFFu, flips, o);
            if (lane == 0) s_flips[warp] = flips;
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned long long t = 0;
#pragma unroll
                for (int w2 = 0; w2 < kQmpWarps; ++w2) t += s_flips[w2];
                s_flip_total[par] = t;
                if (blockIdx.x == 0 && d_cur.flip_bits != nullptr) *d_cur.flip_bits = 0ull;
                QmpSlot* sl = slots + static_cast<size_t>(m) * gridDim.x + blockIdx.x;
                sl->partial = mine;
                __threadfence();
                // diagnostics (sbn_set_wait_test): the last CTA keeps its tag to itself, so every CTA's
                // bounded wait for that slot runs out
                if (!(test_withhold_slot && blockIdx.x == gridDim.x - 1))
                    *reinterpret_cast<volatile unsigned long long*>(&sl->nonce) = nonce;
            }
            __syncthreads();
        }
        // ---- exchange + fix-up of matrix m-1 (published one phase ago by every CTA)
        if (m >= 1) {
            const int par = (m - 1) & 1;
            const QmpSlot* base = slots + static_cast<size_t>(m - 1) * gridDim.x;
            double other = 0.0;
            if (threadIdx.x < gridDim.x) {
                const volatile unsigned long long* flag = &base[threadIdx.x].nonce;
                const unsigned long long t0 = global_timer_ns_qmp();
                unsigned int spins = 0;
                bool seen = (*flag == nonce);
                while (!seen) {
                    seen = (*flag == nonce);
                    if (!seen && ((++spins & 0xFFu) == 0) &&
                        global_timer_ns_qmp() - t0 > *reinterpret_cast<volatile unsigned long long*>(&g_wait_limit_ns)) break;
                }
                if (seen) {
                    __threadfence();
                    other = *reinterpret_cast<const volatile double*>(&base[threadIdx.x].partial);
                } else {
                    s_ok = 0;
                    atomicExch(&g_device_status, static_cast<int>(SBN_ERR_TIMEOUT));
                }
            }
            const double S = qmp_block_sum(other, s_warp);      // fixed order: the same bits in every CTA
            if (!s_ok) return;                                   // a peer never arrived: give up cleanly
            if (threadIdx.x == 0 && d_prev.flip_bits != nullptr && s_flip_total[par] != 0ull)
                atomicAdd(d_prev.flip_bits, s_flip_total[par]);
            const double cnt = static_cast<double>(d_prev.num_units) * 128.0;
            const float gamma = static_cast<float>(S / cnt);
            const float scale = fmaxf(gamma, kEps);
            if (threadIdx.x == 0) {
                s_thr = ternary_threshold(scale);
                if (blockIdx.x == 0) *d_prev.w_scale = scale;
            }
            __syncthreads();
            const float thr = s_thr;
            const unsigned int listed = s_list_count[par];
            const bool bracket_ok = s_bracket[par][0] <= thr && thr <= s_bracket[par][1] &&
                                    listed <= static_cast<unsigned int>(kQmpListCap) && d_prev.dense_q == nullptr &&
                                    d_prev.num_units <= (PATTERN == 68 ? (1u << 25) : (1u << 26));   // listed byte offsets are 32-bit
            if (bracket_ok) {
                // every byte not on the list is already final; the listed ones get the exact compare
                const QmpEntry* list = s_list + par * kQmpListCap;
                uint8_t* vb = reinterpret_cast<uint8_t*>(d_prev.vals);
                for (unsigned int e = threadIdx.x; e < listed; e += kQmpThreads) {
                    const float w = list[e].w;
                    vb[list[e].byte_off] = static_cast<uint8_t>(fabsf(w) >= thr ? (w < 0.0f ? 0xFFu : 0x01u) : 0u);
                }
            } else {
                unsigned int unused = 0;
                if (d_prev.w_bf16) qmp68_pass<true, true>(d_prev, rg_prev, thr, thr, nullptr, nullptr, s_warp, unused);
                else qmp68_pass<false, true>(d_prev, rg_prev, thr, thr, nullptr, nullptr, s_warp, unused);
            }
            __syncthreads();                                     // s_thr / this list may be reused
        }
        d_prev = d_cur;
        rg_prev = rg_cur;
    }
    // every CTA has published its last slot (CTA 0 has just read them all), hence has read the generation
    if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<volatile unsigned long long*>(generation) = gen0 + 1ull;
}

// Copies up to kQmpDescChunk job descriptors, passed by value, into the batch workspace: the batched
// call hands its jobs to the device without a host-side staging copy.
constexpr int kQmpDescChunk = 48;
struct QmpDescChunk {
    QmpDesc d[kQmpDescChunk];
};
static_assert(sizeof(QmpDescChunk) <= 4000, "descriptor chunk must fit the kernel parameter space");
__global__ void __launch_bounds__(64)
qmp_store_descs_kernel(const QmpDescChunk chunk, QmpDesc* __restrict__ dst, int n) {
    pdl_wait();                        // the previous user of the workspace has finished; no early start for successors
    if (threadIdx.x < static_cast<unsigned>(n)) dst[threadIdx.x] = chunk.d[threadIdx.x];
}

// Per-call nonce: unique within the process, low 32 bits never 0.
inline unsigned long long qmp_next_nonce() {
    static std::atomic<unsigned long long> counter{0x5B4E0000ull};
    unsigned long long n = counter.fetch_add(1) + 1;
    if ((n & 0xFFFFFFFFull) == 0ull) n = counter.fetch_add(1) + 1;
    return n;
}

inline QmpDesc qmp_make_desc(const void* W, bool w_bf16, int N, int K, int8_t* vals, uint8_t* meta, float* w_scale,
                             int8_t* dense_q, const uint8_t* prev_meta, unsigned long long* flip_bits,
                             const float* gamma_hint = nullptr) {
    QmpDesc d;
    d.gamma_hint = gamma_hint;
    d.W = W;
    d.w_bf16 = w_bf16 ? 1u : 0u;
    d.vals = reinterpret_cast<uint16_t*>(vals);
    d.meta = meta;
    d.w_scale = w_scale;
    d.dense_q = reinterpret_cast<uint32_t*>(dense_q);
    d.prev_meta = prev_meta;
    d.flip_bits = prev_meta ? flip_bits : nullptr;
    d.num_units = static_cast<uint32_t>(static_cast<size_t>(N) * K / 128);
    d.KB = static_cast<uint32_t>(K / 128);
    return d;
}

// Launch for `count` matrices: `first` by value, the others already copied to `rest_dev`.
template <int PATTERN>
inline sbn_status launch_quantize_mask_pack_batch(const QmpDesc& first, const QmpDesc* rest_dev, int count,
                                                  uint32_t max_units, QmpSlot* slots, unsigned long long* generation,
                                                  cudaStream_t stream) {
    const int test_withhold_slot = g_test_break_waits;
    unsigned long long nonce = qmp_next_nonce();
    // every CTA must be resident at once (they exchange partial sums): never more CTAs than this
    // device has SMs, and never more than the workspace has slots
    const unsigned cap = static_cast<unsigned>(std::min(device_sm_count(), kQmpMaxCtas));
    const unsigned grid = max_units < cap ? max_units : cap;
    static_assert(kQmpThreads >= kQmpMaxCtas, "one thread per slot in the exchange");
    if (!ensure_dynamic_smem<quantize_mask_pack_kernel<PATTERN>>(kQmpSmemBytes)) return SBN_ERR_CUDA;
    // At most one CTA per SM (1024 threads x 64 registers each) and never more CTAs than SMs, so all
    // of them become resident as soon as the SMs are free and the exchange cannot deadlock; if
    // another kernel kept SMs busy for seconds, the bounded wait reports SBN_ERR_TIMEOUT instead.
    const cudaError_t err = launch_kernel(quantize_mask_pack_kernel<PATTERN>, dim3(grid), dim3(kQmpThreads), kQmpSmemBytes, stream,
                                          first, rest_dev, count, slots, generation, nonce, test_withhold_slot);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

}  // namespace sbn
