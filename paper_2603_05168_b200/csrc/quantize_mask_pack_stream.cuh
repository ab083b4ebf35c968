// Part 1 (Eq. 1-3, 2:4 pattern) for one matrix or a batch, as ONE uninterrupted stream over the weights.
//
// quantize_mask_pack.cuh explains the single-read scheme (bracketed threshold, provisional values,
// fix-up list, exact fallback).  What costs time beside the stream itself is latency: the sample that
// brackets the threshold (a round trip to HBM), the exchange of the per-CTA partial sums (two more),
// the fix-up of the listed values, and a handful of CTA-wide barriers per matrix -- 5 to 7 us per
// matrix, a third of a batch of 2B-shaped matrices and more for small ones.  Here none of that stops
// the stream:
//
//   warp 30       the loader: one lane copies the CTA's range of matrix 0, 1, 2, ... into a ring of shared-
//                 memory stages (60 units = 30 KB of fp32 weights each, four stages) with bulk copies that
//                 count their bytes on a stage's `full` barrier; it refills a stage as soon as the 30
//                 computing warps have released it (`empty` barrier).  Three stages are always in flight,
//                 whatever the computing warps are busy with: the loads cost no registers and no issue slots.
//   warps 0..29   pass 1 of matrix 0, 1, 2, ... back to back, stage by stage: a warp takes two units of a
//                 stage (a half-warp per unit, a lane two adjacent groups), always the same ones (fixed order
//                 of additions: the partial sums are reproducible bit for bit); no CTA-wide barrier between
//                 matrices.  A warp leaves its sum |W| and flip count of matrix m in shared memory and
//                 counts itself on `arrived`.
//   warp 31       the finisher.  For matrix m, in this order:
//                   wait until the 30 computing warps have arrived for m, add their sums in a fixed
//                   order, publish {tag, partial} in the workspace;
//                   exchange of matrix m - 1 (published by every CTA one matrix ago, so the slots are
//                   there already), exact gamma, scale, threshold; fix-up of the listed values of
//                   m - 1, or a note that m - 1 needs the exact second pass; its list becomes free;
//                   bracket of matrix m + 2 (from the caller's hint, or from a sample of the matrix that
//                   bulk copies drop into the list just freed).
//                 All of it runs under pass 1 of the following matrices.
//   three lists   matrix m - 1 is being fixed up while m waits and m + 1 is being written; a streaming
//                 warp starts matrix m only once m - 3 is fixed (its list slot is free) and the bracket
//                 of m exists -- both normally long done.
//   tail          after the last matrix every warp joins: exchange and fix-up of the last matrix, then
//                 the exact second passes that were put off (bracket missed, list overflow, or the
//                 dense W_q wanted), all threads working.
//
// Every wait is bounded; one that runs out raises the CTA's abort flag and the device status word.
#pragma once

#include "quantize_mask_pack.cuh"

namespace sbn {

constexpr int kQmpStreamWarps = kQmpWarps - 2;             // 30 compute, warp 30 loads, warp 31 finishes
constexpr int kQmpLoaderWarp = kQmpWarps - 2;
constexpr int kQmpLists = 3;
constexpr int kQmpStreamListCap = 4096;                    // undecided entries per CTA and matrix (see qmp_bracket_from)
constexpr int kQmpStageUnits = 2 * kQmpStreamWarps;        // a half-warp per unit
constexpr int kQmpStages = 4;
constexpr int kQmpStageBytes = kQmpStageUnits * 512;       // fp32 units; bf16 units fill half of a stage
constexpr int kQmpStreamSmemBytes = kQmpStages * kQmpStageBytes + kQmpLists * kQmpStreamListCap * 8;
constexpr int kQmpMaxBatch = 1024;                         // thresholds of put-off second passes live in shared memory

struct QmpStreamShared {
    double warp_sum[kQmpLists][kQmpWarps];
    unsigned int warp_flips[kQmpLists][kQmpWarps];
    unsigned long long flip_total[kQmpLists];
    unsigned int arrived[kQmpLists];                       // streaming warps done with the matrix in this slot
    unsigned int list_count[kQmpLists];
    float bracket[4][2];                                   // [matrix % 4][lo, hi]
    int bracket_upto;                                      // brackets exist for matrices < bracket_upto
    int fixed_upto;                                        // matrices < fixed_upto are finished: their list slot is free
    int abort;
    float thr_tail;
    float thr_second_pass[kQmpMaxBatch];                   // >= 0: this matrix needs the exact second pass with this threshold
    unsigned long long bar_full[kQmpStages];               // a stage's bytes have landed
    unsigned long long bar_empty[kQmpStages];              // the computing warps are done with a stage
    uint32_t ring_issued, ring_used;                       // the loader's copies of this launch, and its ring position
    unsigned long long bar_sample;                         // the finisher's sample has landed
};

// mbarrier and bulk-copy wrappers of the stage ring
__device__ __forceinline__ uint32_t qmp_smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void qmp_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void qmp_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void qmp_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool qmp_mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a barrier phase; gives up (false) when the CTA aborts or the limit runs out.  With
// `drain` it ignores the abort flag: the loader uses it to see its last copies land before the CTA leaves.
__device__ __forceinline__ bool qmp_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, bool drain = false) {
    if (qmp_mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0ull;
    unsigned int spins = 0;
    while (!qmp_mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0u) {
            if (!drain && *abort_flag) return false;
            const unsigned long long now = global_timer_ns_qmp();
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
__device__ __forceinline__ void qmp_bulk_load(uint32_t smem_dst, const void* gmem_src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar) : "memory");
}
// The same for data that is read once (the master weights of pass 1): the lines are the first to leave the
// L2 again, so the stream does not push out what the kernels after this one will read (the packed weights
// this kernel writes, the activations).
__device__ __forceinline__ unsigned long long qmp_policy_evict_first() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void qmp_bulk_load_once(uint32_t smem_dst, const void* gmem_src, uint32_t bytes, uint32_t bar, unsigned long long policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ float4 qmp_lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
// Position in the ring: the number of stages used so far gives the stage and the parity of its current use.
static_assert((kQmpStages & (kQmpStages - 1)) == 0, "stage = count mod kQmpStages by masking");
struct QmpRing {
    uint32_t used;
    __device__ __forceinline__ uint32_t stage() const { return used & (kQmpStages - 1); }
    __device__ __forceinline__ uint32_t phase() const { return (used / kQmpStages) & 1u; }
    __device__ __forceinline__ void advance() { ++used; }
};

// Matrix m of the batch: the first kQmpInlineDescs travel with the launch (kernel parameters: a batch
// that small needs no kernel that stores its descriptors first), `rest` holds 1, 2, ... in global memory.
constexpr int kQmpInlineDescs = 8;
struct QmpInlineDescs {
    QmpDesc d[kQmpInlineDescs];
};
struct QmpBatch {
    const QmpInlineDescs& inl;
    const QmpDesc* rest;
};
__device__ __forceinline__ QmpDesc qmp_desc_of(const QmpBatch& b, int m) {
    return m < kQmpInlineDescs ? b.inl.d[m] : b.rest[m - 1];
}

// Bounded wait for a shared-memory word (written by another warp of this CTA) to reach `want`.
__device__ __forceinline__ bool qmp_wait_ge(volatile int* word, int want, volatile int* abort_flag) {
    if (*word >= want) return true;
    unsigned long long t0 = 0ull;
    unsigned int spins = 0;
    while (*word < want) {
        __nanosleep(64);
        if ((++spins & 0x3Fu) == 0u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns_qmp();
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

// lo / hi of the bracket around the threshold that gamma_est predicts (see quantize_mask_pack.cuh).  An
// estimate from the caller (the scale of the previous training step, Sec. 2.2: the weights move by a
// learning-rate-sized step) gets a bracket six times narrower than one from a sample: almost no warp then
// meets an undecided value, and listing them is a tenth of pass 1's instructions otherwise.  A hint that
// is off by more than that costs the exact second pass, never the result.
constexpr float kQmpBracketHint = 0.005f;
__device__ __forceinline__ void qmp_bracket_from(float gamma_est, uint32_t num_units, bool from_hint, float& lo, float& hi, bool wide = false) {
    const float b = from_hint ? kQmpBracketHint : ((wide || num_units < kQmpSmallMatrixUnits) ? kQmpBracketSmall : kQmpBracket);
    lo = 0.5f * fmaxf(gamma_est * (1.0f - b), kEps) * (1.0f - 1e-6f);
    hi = 0.5f * fmaxf(gamma_est * (1.0f + b), kEps) * (1.0f + 1e-6f);
}

// The caller's estimate of gamma, if it gave a usable one.
__device__ __forceinline__ bool qmp_hint_usable(float g) { return g > 0.0f && g < 3.0e38f; }
__device__ __forceinline__ bool qmp_hint(const QmpDesc& d, float& g) {
    if (d.gamma_hint == nullptr) return false;
    g = *reinterpret_cast<const volatile float*>(d.gamma_hint);
    return qmp_hint_usable(g);
}

// qmp_sample_gamma in two halves, so that something can be started between asking for the sample and using
// it: all of a thread's sample loads are issued (into v), later they are added up over the CTA.
constexpr int kQmpSamplePerWarp = kQmpSampleUnits / kQmpWarps;
__device__ __forceinline__ void qmp_sample_issue(const QmpDesc& d, float4 (&v)[kQmpSamplePerWarp]) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t n_s = qmp_sample_units(d.num_units);
    const uint32_t stride = d.num_units / n_s;
#pragma unroll
    for (int i = 0; i < kQmpSamplePerWarp; ++i) {
        const uint32_t sidx = warp + i * kQmpWarps;
        const uint32_t u = sidx * stride + ((sidx * 2654435761u) >> 8) % stride;
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (sidx < n_s) v[i] = d.w_bf16 ? qmp_load_group<true>(d.W, u, lane) : qmp_load_group<false>(d.W, u, lane);
    }
}
__device__ __forceinline__ float qmp_sample_finish(const QmpDesc& d, const float4 (&v)[kQmpSamplePerWarp], double* s_warp) {
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < kQmpSamplePerWarp; ++i) acc += (fabsf(v[i].x) + fabsf(v[i].y)) + (fabsf(v[i].z) + fabsf(v[i].w));
    const double total = qmp_block_sum(static_cast<double>(acc), s_warp);
    return static_cast<float>(total / (static_cast<double>(qmp_sample_units(d.num_units)) * 128.0));
}

// gamma_est by ONE warp (the finisher, for matrices 1, 2, ... of a batch without hints): the first
// kQmpSampleUnitsSmall of qmp_sample_gamma's scattered units, fetched by bulk copies into `buf` (a list that
// is free at that moment) -- all of them in flight at once, one round trip instead of one per eight units.
// The smaller sample gets the wider bracket (qmp_bracket_from, `wide`).  Returns a negative number if the
// copies did not land within the wait limit (the CTA is then aborting).
constexpr int kQmpSampleUnitsWarp = kQmpSampleUnitsSmall;
static_assert(kQmpSampleUnitsWarp * 512 <= kQmpStreamListCap * 8, "the sample fits a list");
__device__ __forceinline__ float qmp_sample_gamma_warp(const QmpDesc& d, int lane, unsigned char* buf, uint32_t bar, uint32_t& bar_phase,
                                                       volatile int* abort_flag) {
    const uint32_t unit_bytes = d.w_bf16 ? 256u : 512u;
    const uint32_t n_full = qmp_sample_units(d.num_units);
    const uint32_t stride = d.num_units / n_full;
    const uint32_t n_s = min(n_full, static_cast<uint32_t>(kQmpSampleUnitsWarp));
    auto unit_of = [&](uint32_t sidx) { return sidx * stride + ((sidx * 2654435761u) >> 8) % stride; };
    const uint32_t buf_u32 = qmp_smem_u32(buf);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // the list's earlier (generic) use before the copies
    if (lane == 0) qmp_mbar_expect_tx(bar, n_s * unit_bytes);
    __syncwarp();
    for (uint32_t sidx = lane; sidx < n_s; sidx += 32u)
        qmp_bulk_load(buf_u32 + sidx * unit_bytes, static_cast<const char*>(d.W) + static_cast<size_t>(unit_of(sidx)) * unit_bytes, unit_bytes, bar);
    const bool landed = qmp_mbar_wait(bar, bar_phase, abort_flag, true);  // sees its own copies land even if the CTA aborts
    bar_phase ^= 1u;
    if (!landed) return -1.0f;
    float acc = 0.0f;
    const uint32_t chunks = n_s * unit_bytes / 16u;
    for (uint32_t c = lane; c < chunks; c += 32u) {
        const float4 v = qmp_lds128(buf_u32 + c * 16u);
        if (d.w_bf16) {
            const uint32_t r0 = __float_as_uint(v.x), r1 = __float_as_uint(v.y), r2 = __float_as_uint(v.z), r3 = __float_as_uint(v.w);
            acc += ((fabsf(bf16lo_to_f32(r0)) + fabsf(bf16hi_to_f32(r0))) + (fabsf(bf16lo_to_f32(r1)) + fabsf(bf16hi_to_f32(r1)))) +
                   ((fabsf(bf16lo_to_f32(r2)) + fabsf(bf16hi_to_f32(r2))) + (fabsf(bf16lo_to_f32(r3)) + fabsf(bf16hi_to_f32(r3))));
        } else {
            acc += (fabsf(v.x) + fabsf(v.y)) + (fabsf(v.z) + fabsf(v.w));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    __syncwarp();
    return acc / (static_cast<float>(n_s) * 128.0f);
}

// The loader: walks the CTA's ranges of matrix 0, 1, 2, ... stage by stage.  qmp_loader_issue starts up to
// `max_copies` copies (each after its stage has been released) and returns false if a wait ran out.
struct QmpLoader {
    int m;                       // matrix being loaded
    uint32_t u, u_end;           // next unit and end of the CTA's range of it (valid while `open`)
    uint32_t unit_bytes;
    const char* W;
    bool open;
    QmpRing ring;
    uint32_t issued;             // copies of this launch (the drain after an abort needs it)
    unsigned long long policy;   // L2 policy of the copies: read once
};
__device__ __forceinline__ bool qmp_loader_issue(QmpLoader& L, const QmpBatch& batch, int count, uint32_t max_copies,
                                                 uint32_t ring_base, uint32_t bar_full0, uint32_t bar_empty0, volatile int* abort_flag) {
    for (;;) {
        while (!L.open) {
            if (L.m >= count) return true;
            const QmpDesc d = qmp_desc_of(batch, L.m);
            const QmpRange rg = qmp_range(d);
            L.u = rg.u_begin;
            L.u_end = rg.u_end;
            L.unit_bytes = d.w_bf16 ? 256u : 512u;
            L.W = static_cast<const char*>(d.W);
            if (L.u < L.u_end) L.open = true; else ++L.m;
        }
        if (max_copies == 0u) return true;
        --max_copies;
        if (!qmp_mbar_wait(bar_empty0 + 8u * L.ring.stage(), L.ring.phase() ^ 1u, abort_flag)) return false;
        const uint32_t bytes = min(L.u_end - L.u, static_cast<uint32_t>(kQmpStageUnits)) * L.unit_bytes;
        qmp_mbar_expect_tx(bar_full0 + 8u * L.ring.stage(), bytes);
        qmp_bulk_load_once(ring_base + L.ring.stage() * kQmpStageBytes, L.W + static_cast<size_t>(L.u) * L.unit_bytes, bytes, bar_full0 + 8u * L.ring.stage(),
                           L.policy);
        ++L.issued;
        L.ring.advance();
        L.u += kQmpStageUnits;
        if (L.u >= L.u_end) { L.open = false; ++L.m; }
    }
}

// One lane's two groups (32 B of a row) of pass 1: sum |W|, metadata, provisional values, undecided list,
// flip count, as in quantize_mask_pack.cuh.  `meta_row` / `vals_row` point at this lane's byte / word of the
// unit's row inside the metadata and value tiles; `v_off` is the word's byte offset in vals (for the list).
struct QmpPass1Consts {
    float thr_lo, thr_hi, mid, half;
    QmpEntry* list;
    unsigned int* list_count;
};
__device__ __forceinline__ void qmp_pass1_groups(const float4 va, const float4 vb, const QmpPass1Consts& c, uint8_t* meta_row,
                                                 const uint8_t* prev_row, uint32_t* vals_row, uint32_t v_off, double& acc, unsigned int& flips) {
    acc += abs_sum4(va) + abs_sum4(vb);
    float k[4];
    const uint32_t nib0 = select_pair(va, k[0], k[1]);
    const uint32_t nib1 = select_pair(vb, k[2], k[3]);
    if (prev_row != nullptr) {
        const uint32_t prev = *prev_row;
        flips += __popc((nibble_to_mask(nib0) | (nibble_to_mask(nib1) << 4)) ^
                        (nibble_to_mask(prev & 15u) | (nibble_to_mask(prev >> 4) << 4)));
    }
    *meta_row = static_cast<uint8_t>(nib0 | (nib1 << 4));
    *vals_row = ternary_bytes4(k[0], k[1], k[2], k[3], c.thr_hi);
    const float far = fminf(fminf(fabsf(fabsf(k[0]) - c.mid), fabsf(fabsf(k[1]) - c.mid)),
                            fminf(fabsf(fabsf(k[2]) - c.mid), fabsf(fabsf(k[3]) - c.mid)));
    if (far <= c.half) qmp_list_undecided<kQmpStreamListCap>(k, c.thr_lo, c.thr_hi, v_off, c.list, c.list_count);
}

// Pass 1 of one matrix for a computing warp: its two units of every stage of the CTA's range (a half-warp
// per unit, a lane two adjacent groups).  Returns the thread's sum |W|; `ok` turns false if a wait ran out.
template <bool BF16>
__device__ __forceinline__ double qmp_stream_pass1(const QmpDesc& d, const QmpRange rg, const float thr_lo, const float thr_hi,
                                                   QmpEntry* list, unsigned int* list_count, unsigned int& flips,
                                                   QmpRing& ring, uint32_t ring_base, uint32_t bar_full0, uint32_t bar_empty0,
                                                   volatile int* abort_flag, bool& ok) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t l16 = lane & 15;
    const uint32_t KB = d.KB;
    constexpr uint32_t kUnitBytes = BF16 ? 256u : 512u;
    const uint32_t step_n = kQmpStageUnits / KB, step_kb = kQmpStageUnits % KB;
    // |k| in [thr_lo, thr_hi) implies | |k| - mid | <= half (the subtraction is exact, thr_hi < 2 thr_lo;
    // `half` is rounded up by far more than the rounding of `mid`): a cheap test with no false negatives
    const QmpPass1Consts c{thr_lo, thr_hi, 0.5f * (thr_lo + thr_hi), fmaf(thr_hi - thr_lo, 0.50005f, thr_hi * 2.4e-7f), list, list_count};
    double acc = 0.0;
    const uint32_t in_stage = 2u * warp + (lane >> 4);               // this half-warp's unit of every stage
    const uint32_t u_first = rg.u_begin + in_stage;
    uint32_t n_cur = u_first / KB;
    uint32_t kb_cur = u_first - n_cur * KB;
    const uint32_t src_off = ring_base + in_stage * kUnitBytes + l16 * (kUnitBytes / 16u);
    // this lane's place in a row of a metadata tile (byte l16 of 16) and of a value tile (word l16 & 3 of the
    // 16-byte chunk (l16 >> 2) ^ ((row >> 1) & 3), see layouts.cuh)
    uint8_t* const meta_lane = d.meta + l16;
    const uint8_t* const prev_lane = d.prev_meta != nullptr ? d.prev_meta + l16 : nullptr;
    unsigned char* const vals_lane = reinterpret_cast<unsigned char*>(d.vals) + 4u * (l16 & 3u);
    const uint32_t chunk = l16 >> 2;
    const uint32_t range = rg.u_end - rg.u_begin;
    const uint32_t n_stages = (range + kQmpStageUnits - 1) / kQmpStageUnits;
    const uint32_t last_units = range - (n_stages - 1u) * kQmpStageUnits;          // units of the last stage (range > 0)
    for (uint32_t st = 0; st < n_stages; ++st) {
        const uint32_t stage = ring.stage();
        if (!qmp_mbar_wait(bar_full0 + 8u * stage, ring.phase(), abort_flag)) { ok = false; break; }
        const bool mine = st + 1u < n_stages || in_stage < last_units;
        float4 va, vb;
        {
            // a lane without a unit (last stage only) reads what is there: finite or not, it is not used
            const uint32_t src = src_off + stage * kQmpStageBytes;
            if constexpr (BF16) {
                const float4 raw = qmp_lds128(src);
                const uint32_t r0 = __float_as_uint(raw.x), r1 = __float_as_uint(raw.y), r2 = __float_as_uint(raw.z), r3 = __float_as_uint(raw.w);
                va = make_float4(bf16lo_to_f32(r0), bf16hi_to_f32(r0), bf16lo_to_f32(r1), bf16hi_to_f32(r1));
                vb = make_float4(bf16lo_to_f32(r2), bf16hi_to_f32(r2), bf16lo_to_f32(r3), bf16hi_to_f32(r3));
            } else {
                va = qmp_lds128(src);
                vb = qmp_lds128(src + 16u);
            }
        }
        __syncwarp();
        if (lane == 0) qmp_mbar_arrive(bar_empty0 + 8u * stage);           // the values are in registers: the stage may be refilled
        ring.advance();
        const uint32_t tile_idx = (n_cur >> 7) * KB + kb_cur;
        const uint32_t rr = n_cur & 127u;
        n_cur += step_n;
        kb_cur += step_kb;
        if (kb_cur >= KB) { kb_cur -= KB; ++n_cur; }
        if (mine) {
            const size_t m_off = static_cast<size_t>(tile_idx) * 2048u + (rr << 4);
            const size_t v_off = static_cast<size_t>(tile_idx) * 8192u + ((rr << 6) + ((chunk ^ ((rr >> 1) & 3u)) << 4));
            qmp_pass1_groups(va, vb, c, meta_lane + m_off, prev_lane != nullptr ? prev_lane + m_off : nullptr,
                             reinterpret_cast<uint32_t*>(vals_lane + v_off), static_cast<uint32_t>(v_off) + 4u * (l16 & 3u), acc, flips);
        }
    }
    return acc;
}

// What the exact gamma decides for a matrix whose pass 1 is complete: true if the listed values were
// all that had to be redone (and `fix` should run), false if the whole range must be ternarised again.
__device__ __forceinline__ bool qmp_bracket_holds(const QmpDesc& d, float thr, float lo, float hi, unsigned int listed) {
    return lo <= thr && thr <= hi && listed <= static_cast<unsigned int>(kQmpStreamListCap) && d.dense_q == nullptr &&
           d.num_units <= (1u << 26);                        // listed byte offsets are 32-bit
}

__global__ void __launch_bounds__(kQmpThreads, 1)
quantize_mask_pack_stream_kernel(const __grid_constant__ QmpInlineDescs inl, const QmpDesc* __restrict__ rest, int count,
                                 QmpSlot* slots, unsigned long long* generation, unsigned long long call_nonce,
                                 int test_withhold_slot, QmpMemo* memo) {
    extern __shared__ __align__(128) unsigned char s_dyn[];   // [kQmpStages][kQmpStageBytes] ring, then [kQmpLists][kQmpStreamListCap] entries
    QmpEntry* const s_list = reinterpret_cast<QmpEntry*>(s_dyn + kQmpStages * kQmpStageBytes);
    __shared__ QmpStreamShared sh;
    __shared__ double s_warp[kQmpWarps];

    const QmpBatch batch{inl, rest};
    const QmpDesc& first = inl.d[0];
    const QmpDesc& second = inl.d[1];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    volatile int* const abort_flag = &sh.abort;
    const uint32_t ring_base = qmp_smem_u32(s_dyn);
    const uint32_t bar_full0 = qmp_smem_u32(&sh.bar_full[0]), bar_empty0 = qmp_smem_u32(&sh.bar_empty[0]);
    if (threadIdx.x == 0) {
        sh.bracket_upto = 0;
        sh.fixed_upto = 0;
        sh.abort = 0;
        sh.ring_issued = 0u; sh.ring_used = 0u;
        for (int i = 0; i < kQmpLists; ++i) { sh.arrived[i] = 0u; sh.list_count[i] = 0u; sh.flip_total[i] = 0ull; }
        for (int i = 0; i < kQmpStages; ++i) {
            qmp_mbar_init(bar_full0 + 8u * i, 1u);                     // the loader's expect_tx
            qmp_mbar_init(bar_empty0 + 8u * i, kQmpStreamWarps);       // one arrival per computing warp
        }
        qmp_mbar_init(qmp_smem_u32(&sh.bar_sample), 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < kQmpMaxBatch; i += kQmpThreads) sh.thr_second_pass[i] = -1.0f;
    __syncthreads();
    // No early signal to the next kernel of the stream: this kernel writes packed weights, and the
    // GEMM kernels fetch weights before their own dependency wait (see sbn_common.cuh).
    pdl_wait();
    const unsigned long long gen0 = *reinterpret_cast<volatile unsigned long long*>(generation);
    const unsigned long long tag = qmp_tag(call_nonce, gen0);

    // ---- What the first bracket needs is asked for BEFORE the loader fills the ring: the hints of matrices
    // 0 and 1 (4-byte reads) or, without a usable hint, the sample of matrix 0 (all threads, one round
    // trip).  Issued together with the ring's first copies they queue behind the 17 MB that the loaders of
    // all CTAs ask for at the same moment (up to 3.5 us measured, and the CTA that is served last finishes
    // last); so the loader waits for the hints to be there, or for the sample loads to be on their way.
    float g01[2];                                            // both reads in flight before either is looked at
    g01[0] = first.gamma_hint != nullptr ? *reinterpret_cast<const volatile float*>(first.gamma_hint) : 0.0f;
    g01[1] = (count > 1 && second.gamma_hint != nullptr) ? *reinterpret_cast<const volatile float*>(second.gamma_hint) : 0.0f;
    if (memo != nullptr && first.gamma_hint == nullptr) {
        // a single matrix without a hint: what the previous call on this workspace left, if it was this matrix
        // (two 16-byte reads in flight together, not four dependent ones)
        unsigned long long m_tag, m_w;
        uint32_t m_units, m_scale;
        asm volatile("ld.volatile.global.v2.u64 {%0, %1}, [%2];" : "=l"(m_tag), "=l"(m_w) : "l"(memo));
        asm volatile("ld.volatile.global.v2.u32 {%0, %1}, [%2];" : "=r"(m_units), "=r"(m_scale) : "l"(&memo->num_units));
        if (m_tag == kQmpMemoMagic && m_w == reinterpret_cast<unsigned long long>(first.W) && m_units == first.num_units)
            g01[0] = __uint_as_float(m_scale);
    }
    const bool hinted01[2] = {qmp_hint_usable(g01[0]), qmp_hint_usable(g01[1])};
    float4 sample0[kQmpSamplePerWarp];
    if (!hinted01[0]) qmp_sample_issue(first, sample0);
    QmpLoader loader{0, 0u, 0u, 0u, nullptr, false, QmpRing{0u}, 0u, qmp_policy_evict_first()};
    const bool is_loader = warp == kQmpLoaderWarp && lane == 0;
    if (is_loader) qmp_loader_issue(loader, batch, count, kQmpStages, ring_base, bar_full0, bar_empty0, abort_flag);
    if (!hinted01[0]) g01[0] = qmp_sample_finish(first, sample0, s_warp);
    if (threadIdx.x == 0) {
        qmp_bracket_from(g01[0], first.num_units, hinted01[0], sh.bracket[0][0], sh.bracket[0][1]);
        // matrix 1: from its hint here; without one the finisher samples it while matrix 0 streams
        if (hinted01[1]) qmp_bracket_from(g01[1], second.num_units, true, sh.bracket[1][0], sh.bracket[1][1]);
        sh.bracket_upto = hinted01[1] ? 2 : 1;
    }
    __syncthreads();

    if (warp < kQmpStreamWarps) {
        // ------------------------------------------------------------------ computing warps
        QmpRing ring{0u};
        for (int m = 0; m < count; ++m) {
            const int slot = m % kQmpLists;
            if (!qmp_wait_ge(&sh.bracket_upto, m + 1, abort_flag)) break;
            if (!qmp_wait_ge(&sh.fixed_upto, m - (kQmpLists - 1), abort_flag)) break;
            const QmpDesc d = qmp_desc_of(batch, m);
            const QmpRange rg = qmp_range(d);
            const float lo = *reinterpret_cast<volatile float*>(&sh.bracket[m & 3][0]);
            const float hi = *reinterpret_cast<volatile float*>(&sh.bracket[m & 3][1]);
            unsigned int flips = 0;
            bool ok = true;
            double mine = d.w_bf16 ? qmp_stream_pass1<true>(d, rg, lo, hi, s_list + slot * kQmpStreamListCap, &sh.list_count[slot], flips,
                                                            ring, ring_base, bar_full0, bar_empty0, abort_flag, ok)
                                   : qmp_stream_pass1<false>(d, rg, lo, hi, s_list + slot * kQmpStreamListCap, &sh.list_count[slot], flips,
                                                             ring, ring_base, bar_full0, bar_empty0, abort_flag, ok);
            if (!ok) break;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
                flips += __shfl_xor_sync(0xFFFFFFFFu, flips, o);
            }
            __syncwarp();                                    // every lane's list entries are written
            if (lane == 0) {
                sh.warp_sum[slot][warp] = mine;
                sh.warp_flips[slot][warp] = flips;
                __threadfence_block();                       // the sums, and this warp's list entries, before the count
                atomicAdd(&sh.arrived[slot], 1u);
            }
            __syncwarp();
        }
    } else if (warp == kQmpLoaderWarp) {
        // ------------------------------------------------------------------ the loader (warp 30, one lane)
        if (is_loader) {
            qmp_loader_issue(loader, batch, count, 0xFFFFFFFFu, ring_base, bar_full0, bar_empty0, abort_flag);
            sh.ring_issued = loader.issued;                  // for the drain, should the CTA abort
            sh.ring_used = loader.ring.used;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ the finisher (warp 31)
        bool ok = true;
        uint32_t sample_phase = 0u;
        if (count > 1 && !hinted01[1]) {
            // bracket of matrix 1 from a sample into its own (still unused) list, while matrix 0 streams
            const float g = qmp_sample_gamma_warp(second, lane, reinterpret_cast<unsigned char*>(s_list + 1 * kQmpStreamListCap),
                                                  qmp_smem_u32(&sh.bar_sample), sample_phase, abort_flag);
            if (g < 0.0f) {
                ok = false;
            } else {
                if (lane == 0) {
                    qmp_bracket_from(g, second.num_units, false, sh.bracket[1][0], sh.bracket[1][1], true);
                    __threadfence_block();
                    *reinterpret_cast<volatile int*>(&sh.bracket_upto) = 2;
                }
                __syncwarp();
            }
        }
        for (int m = 0; ok && m < count; ++m) {
            const int slot = m % kQmpLists;
            // bracket of matrix m + 2 from the caller's hint, well before the computing warps ask for it
            bool sample_next = false;
            if (m + 2 < count) {
                const QmpDesc d2 = qmp_desc_of(batch, m + 2);
                float g;
                if (qmp_hint(d2, g)) {
                    if (lane == 0) {
                        qmp_bracket_from(g, d2.num_units, true, sh.bracket[(m + 2) & 3][0], sh.bracket[(m + 2) & 3][1]);
                        __threadfence_block();
                        *reinterpret_cast<volatile int*>(&sh.bracket_upto) = m + 3;
                    }
                    __syncwarp();
                } else {
                    sample_next = true;
                }
            }
            // matrix m: every streaming warp has arrived -> this CTA's partial sum, published
            if (!qmp_wait_ge(reinterpret_cast<volatile int*>(&sh.arrived[slot]), kQmpStreamWarps, abort_flag)) { ok = false; break; }
            __threadfence_block();
            const QmpDesc d = qmp_desc_of(batch, m);
            {
                double v = lane < kQmpStreamWarps ? *reinterpret_cast<volatile double*>(&sh.warp_sum[slot][lane]) : 0.0;
                unsigned int f = lane < kQmpStreamWarps ? *reinterpret_cast<volatile unsigned int*>(&sh.warp_flips[slot][lane]) : 0u;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                    f += __shfl_xor_sync(0xFFFFFFFFu, f, o);
                }
                if (lane == 0) {
                    sh.flip_total[slot] = f;
                    if (blockIdx.x == 0 && d.flip_bits != nullptr) *d.flip_bits = 0ull;
                    QmpSlot* sl = slots + static_cast<size_t>(m) * gridDim.x + blockIdx.x;
                    sl->partial = v;
                    __threadfence();
                    if (!(test_withhold_slot && blockIdx.x == gridDim.x - 1))
                        *reinterpret_cast<volatile unsigned long long*>(&sl->nonce) = tag;
                }
                __syncwarp();
            }
            // matrix m - 1: exchange, exact threshold, fix-up
            if (m >= 1) {
                const int pslot = (m - 1) % kQmpLists;
                const QmpDesc dp = qmp_desc_of(batch, m - 1);
                const QmpSlot* base = slots + static_cast<size_t>(m - 1) * gridDim.x;
                // a lane looks after the slots lane, lane + 32, ...: all its flags are polled together, then all
                // its partial sums are read together (two round trips in all, not two per slot)
                constexpr int kPerLane = (kQmpMaxCtas + 31) / 32;
                {
                    unsigned long long t0 = 0ull;
                    unsigned int spins = 0;
                    bool seen = false;
                    while (!seen) {
                        seen = true;
#pragma unroll
                        for (int j = 0; j < kPerLane; ++j) {
                            const unsigned int i = lane + 32u * j;
                            if (i < gridDim.x) seen = seen && (*reinterpret_cast<const volatile unsigned long long*>(&base[i].nonce) == tag);
                        }
                        if (!seen && ((++spins & 0xFFu) == 0u)) {
                            if (*abort_flag) break;
                            const unsigned long long now = global_timer_ns_qmp();
                            if (t0 == 0ull) t0 = now;
                            else if (now - t0 > *reinterpret_cast<volatile unsigned long long*>(&g_wait_limit_ns)) break;
                        }
                    }
                    if (!seen) ok = false;
                }
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) {
                    if (lane == 0) { *abort_flag = 1; atomicExch(&g_device_status, static_cast<int>(SBN_ERR_TIMEOUT)); }
                    break;
                }
                __threadfence();
                double part[kPerLane];
#pragma unroll
                for (int j = 0; j < kPerLane; ++j) {
                    const unsigned int i = lane + 32u * j;
                    part[j] = i < gridDim.x ? *reinterpret_cast<const volatile double*>(&base[i].partial) : 0.0;
                }
                double sum = 0.0;
#pragma unroll
                for (int j = 0; j < kPerLane; ++j) sum += part[j];                 // a lane's slots in increasing order
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);    // the same order in every CTA
                const float gamma = static_cast<float>(sum / (static_cast<double>(dp.num_units) * 128.0));
                const float scale = fmaxf(gamma, kEps);
                float thr = 0.0f;
                if (lane == 0) {
                    thr = ternary_threshold(scale);
                    if (blockIdx.x == 0) *dp.w_scale = scale;
                    if (dp.flip_bits != nullptr && sh.flip_total[pslot] != 0ull) atomicAdd(dp.flip_bits, sh.flip_total[pslot]);
                }
                thr = __shfl_sync(0xFFFFFFFFu, thr, 0);
                const unsigned int listed = *reinterpret_cast<volatile unsigned int*>(&sh.list_count[pslot]);
                if (qmp_bracket_holds(dp, thr, sh.bracket[(m - 1) & 3][0], sh.bracket[(m - 1) & 3][1], listed)) {
                    const QmpEntry* list = s_list + pslot * kQmpStreamListCap;
                    uint8_t* vb = reinterpret_cast<uint8_t*>(dp.vals);
                    for (unsigned int e = lane; e < listed; e += 32u) {
                        const float w = list[e].w;
                        vb[list[e].byte_off] = static_cast<uint8_t>(fabsf(w) >= thr ? (w < 0.0f ? 0xFFu : 0x01u) : 0u);
                    }
                } else if (lane == 0) {
                    sh.thr_second_pass[m - 1] = thr;
                }
                __syncwarp();
                if (lane == 0) {
                    sh.arrived[pslot] = 0u;
                    sh.list_count[pslot] = 0u;
                    __threadfence_block();
                    *reinterpret_cast<volatile int*>(&sh.fixed_upto) = m;
                }
                __syncwarp();
            }
            // bracket of matrix m + 2 from a sample, if it has no hint: a whole matrix before the computing warps
            // ask for it.  The sample lands in the list that matrix m - 1 has just given back (the one m + 2 will use).
            if (sample_next) {
                const QmpDesc d2 = qmp_desc_of(batch, m + 2);
                const float g = qmp_sample_gamma_warp(d2, lane, reinterpret_cast<unsigned char*>(s_list + ((m + 2) % kQmpLists) * kQmpStreamListCap),
                                                      qmp_smem_u32(&sh.bar_sample), sample_phase, abort_flag);
                if (g < 0.0f) { ok = false; break; }
                if (lane == 0) {
                    qmp_bracket_from(g, d2.num_units, false, sh.bracket[(m + 2) & 3][0], sh.bracket[(m + 2) & 3][1], true);
                    __threadfence_block();
                    *reinterpret_cast<volatile int*>(&sh.bracket_upto) = m + 3;
                }
                __syncwarp();
            }
        }
    }
    __syncthreads();
    if (sh.abort) {
        // No bulk copy may still be writing this CTA's shared memory when it leaves: the last
        // min(issued, kQmpStages) copies are the ones that can be in flight; the ring position points past the newest.
        if (threadIdx.x == 0) {
            QmpRing ring{sh.ring_used};
            const uint32_t back = min(sh.ring_issued, static_cast<uint32_t>(kQmpStages));
            for (uint32_t j = 0; j < back; ++j) {
                --ring.used;
                qmp_mbar_wait(bar_full0 + 8u * ring.stage(), ring.phase(), abort_flag, true);
            }
        }
        return;
    }

    // ---- tail: the last matrix, all threads
    {
        const int m = count - 1;
        const int slot = m % kQmpLists;
        const QmpDesc d = qmp_desc_of(batch, m);
        const QmpRange rg = qmp_range(d);
        const QmpSlot* base = slots + static_cast<size_t>(m) * gridDim.x;
        double other = 0.0;
        if (threadIdx.x < gridDim.x) {
            const volatile unsigned long long* flag = &base[threadIdx.x].nonce;
            unsigned long long t0 = 0ull;
            unsigned int spins = 0;
            bool seen = (*flag == tag);
            while (!seen) {
                seen = (*flag == tag);
                if (!seen && ((++spins & 0xFFu) == 0u)) {
                    const unsigned long long now = global_timer_ns_qmp();
                    if (t0 == 0ull) t0 = now;
                    else if (now - t0 > *reinterpret_cast<volatile unsigned long long*>(&g_wait_limit_ns)) break;
                }
            }
            if (seen) {
                __threadfence();
                other = *reinterpret_cast<const volatile double*>(&base[threadIdx.x].partial);
            } else {
                sh.abort = 1;
                atomicExch(&g_device_status, static_cast<int>(SBN_ERR_TIMEOUT));
            }
        }
        const double S = qmp_block_sum(other, s_warp);          // fixed order: the same bits in every CTA
        if (sh.abort) return;                                    // a peer never arrived: give up cleanly
        if (threadIdx.x == 0 && d.flip_bits != nullptr && sh.flip_total[slot] != 0ull) atomicAdd(d.flip_bits, sh.flip_total[slot]);
        const float gamma = static_cast<float>(S / (static_cast<double>(d.num_units) * 128.0));
        const float scale = fmaxf(gamma, kEps);
        if (threadIdx.x == 0) {
            sh.thr_tail = ternary_threshold(scale);
            if (blockIdx.x == 0) *d.w_scale = scale;
        }
        __syncthreads();
        const float thr = sh.thr_tail;
        const unsigned int listed = sh.list_count[slot];
        if (qmp_bracket_holds(d, thr, sh.bracket[m & 3][0], sh.bracket[m & 3][1], listed)) {
            const QmpEntry* list = s_list + slot * kQmpStreamListCap;
            uint8_t* vb = reinterpret_cast<uint8_t*>(d.vals);
            for (unsigned int e = threadIdx.x; e < listed; e += kQmpThreads) {
                const float w = list[e].w;
                vb[list[e].byte_off] = static_cast<uint8_t>(fabsf(w) >= thr ? (w < 0.0f ? 0xFFu : 0x01u) : 0u);
            }
        } else {
            if (d.w_bf16) qmp_pass2_full<true>(d, rg, thr);
            else qmp_pass2_full<false>(d, rg, thr);
        }
    }
    // ---- the second passes that were put off
    for (int m = 0; m + 1 < count; ++m) {
        const float thr = sh.thr_second_pass[m];
        if (thr >= 0.0f) {
            const QmpDesc d = qmp_desc_of(batch, m);
            const QmpRange rg = qmp_range(d);
            if (d.w_bf16) qmp_pass2_full<true>(d, rg, thr);
            else qmp_pass2_full<false>(d, rg, thr);
        }
    }
    // every CTA has published its last slot (CTA 0 has just read them all), hence has read the generation
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *reinterpret_cast<volatile unsigned long long*>(generation) = gen0 + 1ull;
        if (memo != nullptr) {
            // every CTA has read the memo by now (they have all published since)
            memo->W = first.W;
            memo->num_units = first.num_units;
            memo->scale = *reinterpret_cast<volatile float*>(first.w_scale);     // written by this thread above
            __threadfence();
            memo->magic = kQmpMemoMagic;
        }
    }
}

// Launch for `count` (<= kQmpMaxBatch) matrices: the first kQmpInlineDescs of `descs_host` by value, matrices
// 1, 2, ... already copied to `rest_dev` if there are more than that.
inline sbn_status launch_quantize_mask_pack_stream(const QmpDesc* descs_host, const QmpDesc* rest_dev, int count,
                                                   uint32_t max_units, QmpSlot* slots, unsigned long long* generation,
                                                   cudaStream_t stream, QmpMemo* memo = nullptr) {
    QmpInlineDescs inl;
    for (int i = 0; i < kQmpInlineDescs; ++i) inl.d[i] = descs_host[i < count ? i : 0];
    const int test_withhold_slot = g_test_break_waits;
    const unsigned long long nonce = qmp_next_nonce();
    // every CTA must be resident at once (they exchange partial sums): never more CTAs than this
    // device has SMs, and never more than the workspace has slots
    const unsigned cap = static_cast<unsigned>(std::min(device_sm_count(), kQmpMaxCtas));
    const unsigned grid = max_units < cap ? max_units : cap;
    if (!ensure_dynamic_smem<quantize_mask_pack_stream_kernel>(kQmpStreamSmemBytes)) return SBN_ERR_CUDA;
    // At most one CTA per SM (1024 threads x 64 registers each) and never more CTAs than SMs, so all
    // of them become resident as soon as the SMs are free and the exchange cannot deadlock; if
    // another kernel kept SMs busy for seconds, the bounded wait reports SBN_ERR_TIMEOUT instead.
    const cudaError_t err = launch_kernel(quantize_mask_pack_stream_kernel, dim3(grid), dim3(kQmpThreads), kQmpStreamSmemBytes, stream,
                                          inl, rest_dev, count, slots, generation, nonce, test_withhold_slot, count == 1 ? memo : nullptr);
    ++g_launch_count;
    return err == cudaSuccess ? SBN_OK : SBN_ERR_CUDA;
}

inline sbn_status launch_quantize_mask_pack(const void* W, bool w_bf16, int N, int K, int8_t* vals,
                                            uint8_t* meta, float* w_scale, int8_t* dense_q,
                                            const uint8_t* prev_meta,
                                            unsigned long long* flip_bits, QmpWorkspace* ws,
                                            cudaStream_t stream) {
    const QmpDesc d = qmp_make_desc(W, w_bf16, N, K, vals, meta, w_scale, dense_q, prev_meta, flip_bits);
    return launch_quantize_mask_pack_stream(&d, nullptr, 1, d.num_units, ws->slot, &ws->generation, stream, &ws->memo);
}

}  // namespace sbn
