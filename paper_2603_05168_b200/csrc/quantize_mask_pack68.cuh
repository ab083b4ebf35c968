// The 6:8 pattern (Sec. 2.2: of every 8 consecutive input weights the 6 largest |w| are kept; the
// pattern of the paper's main results) on tensor cores that only know 2:4.
//
// Three overlapping 4-column windows cover a group of 8 columns:
//     window 0 = columns 0..3,   window 1 = columns 2..5,   window 2 = columns 4..7.
// Whatever 6 columns a group keeps, they can be dealt out so that every window holds exactly two
// of them (at most two columns are missing, so columns 0..3 keep >= 2 and 4..7 keep >= 2: window 0
// takes what is kept of {0,1} and fills up from {2,3}, window 2 takes what is kept of {6,7} and
// fills up from {4,5}, and exactly two kept columns of {2..5} remain for window 1).  A 6:8 matrix
// [N][K] is therefore a 2:4 matrix [N][K' = 3K/2] over activations whose rows are expanded the
// same way (K' column 12 g + 4 w + s  <-  column 8 g + 2 w + s; see quant_act.cuh), and the
// sparse GEMM runs unchanged at 3/4 of the dense MMA work.  The outputs are the compressed values
// and metadata of that [N][K'] matrix in the tiled layouts of layouts.cuh.
//
// Same single-pass scheme as the 2:4 kernel (sample -> bracket, pass 1 with provisional
// ternarisation and a list of undecided kept values, exchange of partial sums, fix-up).  A lane
// owns one group of 8 (32 B of a row): 6 bytes of values (three 2-byte stores) and 12 bits of
// metadata (a quad of lanes writes its 6 bytes as three 2-byte stores).
#pragma once

#include "quantize_mask_pack.cuh"

namespace sbn {

// Eq. 2 for one group of 8: bit j set = column j kept.  The two smallest |w| are dropped; among
// equal magnitudes the higher column goes first (the lower column wins a tie, as in the 2:4 rule).
__device__ __forceinline__ uint32_t select6of8(const float (&a)[8]) {
    float m = a[7];
    int i1 = 7;
#pragma unroll
    for (int i = 6; i >= 0; --i) {
        if (a[i] < m) { m = a[i]; i1 = i; }
    }
    float m2 = (i1 == 7) ? __int_as_float(0x7F800000) : a[7];
    int i2 = 7;
#pragma unroll
    for (int i = 6; i >= 0; --i) {
        const float b = (i == i1) ? __int_as_float(0x7F800000) : a[i];
        if (b < m2) { m2 = b; i2 = i; }
    }
    return 0xFFu ^ (1u << i1) ^ (1u << i2);
}

// Deals the kept columns S (6 bits set of 8) out to the three windows: 4-bit masks, two bits each.
__device__ __forceinline__ void windows68(uint32_t S, uint32_t& m0, uint32_t& m1, uint32_t& m2) {
    const uint32_t L = S & 3u, ML = (S >> 2) & 3u, MR = (S >> 4) & 3u, R = (S >> 6) & 3u;
    const uint32_t need_l = 2u - __popc(L);
    const uint32_t take_l = need_l == 0u ? 0u : (need_l == 1u ? (ML & (0u - ML)) : ML);        // lowest first
    const uint32_t need_r = 2u - __popc(R);
    const uint32_t take_r = need_r == 0u ? 0u : (need_r == 1u ? (MR == 3u ? 2u : MR) : MR);    // highest first
    m0 = L | (take_l << 2);
    m2 = take_r | (R << 2);
    m1 = (ML & ~take_l) | ((MR & ~take_r) << 2);
}

// 2:4 metadata nibble (i0 | i1 << 2, i0 < i1) of a 4-bit mask with exactly two bits set.
__device__ __forceinline__ uint32_t mask4_to_nibble(uint32_t m) {
    constexpr uint32_t kLo = (4u << 12) | (8u << 20) | (9u << 24);      // masks 3, 5, 6
    constexpr uint32_t kHi = (12u << 4) | (13u << 8) | (14u << 16);     // masks 9, 10, 12
    return (((m & 8u) ? kHi : kLo) >> (4u * (m & 7u))) & 15u;
}
// The two kept weights of a window in column order.
__device__ __forceinline__ void window_values(uint32_t m, float c0, float c1, float c2, float c3, float& v0, float& v1) {
    v0 = (m & 1u) ? c0 : ((m & 2u) ? c1 : c2);
    v1 = (m & 8u) ? c3 : ((m & 4u) ? c2 : c1);
}

// Kept-column mask of a group of 8 from its three metadata nibbles.
__device__ __forceinline__ uint32_t mask8_from_meta12(uint32_t m12) {
    return nibble_to_mask(m12 & 15u) | (nibble_to_mask((m12 >> 4) & 15u) << 2) | (nibble_to_mask((m12 >> 8) & 15u) << 4);
}

// byte offset in the tiled metadata of byte column b of row n (K' space, KBp = K'/128)
__device__ __forceinline__ size_t meta68_offset(uint32_t n, uint32_t b, uint32_t KBp) {
    return (static_cast<size_t>(n >> 7) * KBp + (b >> 4)) * 2048u + ((n & 127u) << 4) + (b & 15u);
}
// byte offset in the tiled values of compressed byte column c of row n
__device__ __forceinline__ size_t vals68_offset(uint32_t n, uint32_t c, uint32_t KBp) {
    return (static_cast<size_t>(n >> 7) * KBp + (c >> 6)) * 8192u + vals_in_tile(n & 127u, c & 63u);
}

// Pass over this CTA's range.  FINAL = false: pass 1 (sum |W|, metadata, flip count, provisional
// values against thr_hi, list of the kept values in [thr_lo, thr_hi)).  FINAL = true: the values
// again with the exact threshold (thr_hi = thr), nothing else.
template <bool BF16, bool FINAL>
__device__ __forceinline__ double qmp68_pass(const QmpDesc& d, const QmpRange rg, const float thr_lo, const float thr_hi,
                                             QmpEntry* list, unsigned int* list_count, double* s_warp,
                                             unsigned int& flips) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t l16 = lane & 15;
    const uint32_t quad_lane = l16 & 3u;
    const uint32_t KB = d.KB;
    const uint32_t KBp = KB + (KB >> 1);                      // K' / 128
    constexpr uint32_t kStep = 2 * kQmpWarps;
    constexpr uint32_t kUnitBytes = BF16 ? 256u : 512u;
    const bool count_flips = !FINAL && d.prev_meta != nullptr;
    uint8_t* vals_b = reinterpret_cast<uint8_t*>(d.vals);
    double acc = 0.0;
    const uint32_t u_first = rg.u_begin + 2 * warp + (lane >> 4);
    const uint32_t step_n = kStep / KB, step_kb = kStep % KB;  // a thread's next unit, without a division
    uint32_t n = u_first / KB;
    uint32_t kb = u_first - n * KB;
    if (threadIdx.x == 0) {
        for (int j = 1; j < kQmpPrefetchAhead; ++j) {
            const uint32_t ub = rg.u_begin + j * kStep;
            if (ub < rg.u_end) prefetch_l2_bulk(static_cast<const char*>(d.W) + static_cast<size_t>(ub) * kUnitBytes, min(rg.u_end - ub, kStep) * kUnitBytes);
        }
    }
    for (uint32_t u0 = rg.u_begin; u0 < rg.u_end; u0 += kStep, n += step_n, kb += step_kb) {
        if (kb >= KB) { kb -= KB; ++n; }
        if (threadIdx.x == 0) {
            const uint32_t ub = u0 + kQmpPrefetchAhead * kStep;
            if (ub < rg.u_end) prefetch_l2_bulk(static_cast<const char*>(d.W) + static_cast<size_t>(ub) * kUnitBytes, min(rg.u_end - ub, kStep) * kUnitBytes);
        }
        const uint32_t uq = u0 + (u_first - rg.u_begin);
        const bool active = uq < rg.u_end;                     // uniform over a half-warp
        float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vb = va;
        if (active) qmp_load_group_pair<BF16>(d.W, uq, l16, va, vb);
        if constexpr (!FINAL) acc += abs_sum4(va) + abs_sum4(vb);
        const uint32_t g_row = kb * 16u + l16;                 // group of 8 within the row
        const float w[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
        float a[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = fabsf(w[i]);
        const uint32_t S = select6of8(a);
        uint32_t m0, m1, m2;
        windows68(S, m0, m1, m2);
        float k[6];
        window_values(m0, w[0], w[1], w[2], w[3], k[0], k[1]);
        window_values(m1, w[2], w[3], w[4], w[5], k[2], k[3]);
        window_values(m2, w[4], w[5], w[6], w[7], k[4], k[5]);
        if constexpr (!FINAL) {
            const uint32_t m12 = mask4_to_nibble(m0) | (mask4_to_nibble(m1) << 4) | (mask4_to_nibble(m2) << 8);
            if (count_flips) {
                // this group's 12 bits of the previous metadata: bits 12 g .. 12 g + 11 of the row.
                // meta may be the same buffer as prev_meta: every byte a quad overwrites below is read
                // here by lanes of that quad only, and the warp barrier orders those reads first.
                if (active) {
                    const uint32_t b0 = (3u * g_row) >> 1;
                    const uint32_t lo = d.prev_meta[meta68_offset(n, b0, KBp)];
                    const uint32_t hi = d.prev_meta[meta68_offset(n, b0 + 1u, KBp)];
                    const uint32_t p12 = ((lo | (hi << 8)) >> ((g_row & 1u) * 4u)) & 0xFFFu;
                    flips += __popc(S ^ mask8_from_meta12(p12));
                }
                __syncwarp();
            }
            // a quad's 48 bits leave as three 2-byte stores (lanes 0..2 of the quad)
            const uint32_t nxt = __shfl_down_sync(0xFFFFFFFFu, m12, 1);
            if (active && quad_lane < 3u) {
                const uint32_t out = ((m12 >> (4u * quad_lane)) | (nxt << (12u - 4u * quad_lane))) & 0xFFFFu;
                const size_t m_off = meta68_offset(n, 6u * (g_row >> 2) + 2u * quad_lane, KBp);
                *reinterpret_cast<uint16_t*>(d.meta + m_off) = static_cast<uint16_t>(out);
            }
        }
        if (active) {
            uint32_t off[3];
            unsigned int cnt = 0;
            bool und[6];
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                off[j] = static_cast<uint32_t>(vals68_offset(n, 6u * g_row + 2u * j, KBp));
                *reinterpret_cast<uint16_t*>(vals_b + off[j]) = static_cast<uint16_t>(ternary_bytes2(k[2 * j], k[2 * j + 1], thr_hi));
            }
            if constexpr (!FINAL) {
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const float ak = fabsf(k[i]);
                    und[i] = ak >= thr_lo && ak < thr_hi;
                    cnt += und[i] ? 1u : 0u;
                }
                if (cnt != 0u) {
                    unsigned int at = atomicAdd(list_count, cnt);
#pragma unroll
                    for (int i = 0; i < 6; ++i) {
                        if (und[i]) {
                            if (at < static_cast<unsigned int>(kQmpListCap)) { list[at].byte_off = off[i >> 1] + (i & 1); list[at].w = k[i]; }
                            ++at;
                        }
                    }
                }
            }
        }
    }
    if constexpr (FINAL) return 0.0;
    else return qmp_block_sum(acc, s_warp);
}

}  // namespace sbn
