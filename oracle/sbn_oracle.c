/*
 * sbn_oracle.c -- CPU oracle for the 2:4-sparse ternary BitLinear path of Sparse-BitNet.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the paper defines.
 * It is called from the tests, from the smoke check and from the benchmark's CPU-baseline leg,
 * and from nowhere else.  It shares no code, header, table or helper with the CUDA library and
 * neither side includes the other.
 *
 * Every function follows one passage of the paper, in the paper's order and notation:
 *   W        latent ("master") weights, d_out x d_in, here N x K row-major fp32     (Sec. 2.1)
 *   gamma    mean absolute value of all entries of W                                 (Eq. 1)
 *   W_q      RoundClip(W / gamma, -1, +1), ternary                                   (Eq. 1)
 *   M_{N:M}  per-group top-N indicator of |W| on the pre-quantised weights           (Eq. 2)
 *   W_eff    W_q (.) M_{N:M}                                                         (Eq. 3)
 *   x~       per-token absmax int8 activations                                       (Sec. 2.1)
 *   y        s * (W_eff x~), s absorbing both quantisation scales                    (Eq. 4)
 *   r_t      mask flip rate                                                          (flip-rate Eq., Sec. 4)
 *
 * Readings taken where the paper is silent or inconsistent (each is also listed in the design
 * notes of the repository):
 *   - epsilon: the pseudo-code of Algorithm 2 clamps both scales from below at 1e-5; that is the
 *     only numeric value the paper gives, so scale = max(gamma, 1e-5) and max|x| -> max(., 1e-5).
 *   - rounding: Algorithm 2 calls round(), i.e. round-half-to-even on fp32 (rintf here).
 *   - gamma is accumulated in double and cast to fp32 once.
 *   - Algorithm 2 divides W by the scale and multiplies x by s_x = 127 / max|x|; both are kept
 *     literally (one IEEE fp32 division, resp. one IEEE fp32 multiplication, no contraction).
 *   - ties in the top-N selection: larger |w| first, equal |w| -> lower column index kept.
 *   - gamma is taken over the whole dense W (Eq. 1 and the "quant-then-mask" bullet of Sec. 4),
 *     not over the masked subset.
 *   - groups are contiguous along d_in (K), aligned to column 0.
 *
 * Compressed 2:4 layout written by sbn_oracle_pack24 (the paper fixes none; this one is the
 * contract of the library):
 *   vals[n][2g], vals[n][2g+1] = W_q at the two kept columns 4g+i0 < 4g+i1 of group g
 *   nibble(g) = i0 | (i1 << 2);  meta[n][b] = nibble(2b) | (nibble(2b+1) << 4)
 *
 * Build: gcc -O2 -fPIC -shared -fopenmp -ffp-contract=off -fno-fast-math
 * OpenMP splits independent rows/tokens only; it never changes an order of summation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SBN_ORACLE_EPS 1e-5f

/* ---------------------------------------------------------------------------------------------
 * Eq. 1 (scale): gamma = ||W||_1 / (d_out * d_in), accumulated in double in row-major order.
 * scale = max(gamma, 1e-5) (Algorithm 2's clamp).
 * near_tie (optional) is set to 1 when the ORDER of the double-precision additions can decide the fp32
 * value of gamma: when a second order (pairwise) does round differently, or when S / D lies within
 * 8 * sqrt(D) * 2^-53 (relative) of the midpoint between two fp32 values -- the typical spread of
 * double-precision sums of D terms taken in different orders.  An implementation that adds the same
 * doubles in an order of its own (a parallel reduction) may then round the other way without being
 * wrong; the caller should reseed instead of reporting a mismatch.
 * ------------------------------------------------------------------------------------------- */
static double pairwise_abs_sum(const float *w, int64_t n)
{
    if (n <= 64) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += fabs((double)w[i]);
        return s;
    }
    int64_t h = n / 2;
    return pairwise_abs_sum(w, h) + pairwise_abs_sum(w + h, n - h);
}

void sbn_oracle_absmean_scale(const float *W, int64_t N, int64_t K,
                              float *gamma_out, float *scale_out, int *near_tie)
{
    const int64_t D = N * K;
    double S = 0.0;
    for (int64_t i = 0; i < D; ++i) S += fabs((double)W[i]);
    float gamma = (D > 0) ? (float)(S / (double)D) : 0.0f;
    if (near_tie) {
        double S2 = pairwise_abs_sum(W, D);
        float g2 = (D > 0) ? (float)(S2 / (double)D) : 0.0f;
        int close = 0;
        if (D > 0 && gamma > 0.0f) {
            const double q = S / (double)D;
            const double tol = 8.0 * sqrt((double)D) * ldexp(1.0, -53) * q;
            const double up = 0.5 * ((double)gamma + (double)nextafterf(gamma, INFINITY));
            const double dn = 0.5 * ((double)gamma + (double)nextafterf(gamma, 0.0f));
            close = (fabs(q - up) <= tol) || (fabs(q - dn) <= tol);
        }
        *near_tie = (g2 != gamma) || close;
    }
    if (gamma_out) *gamma_out = gamma;
    if (scale_out) *scale_out = (gamma > SBN_ORACLE_EPS) ? gamma : SBN_ORACLE_EPS;
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 2 (mask): for every contiguous group of m_group columns keep the n_keep entries with the
 * largest |W|.  Stable selection: repeatedly take the not-yet-taken entry with the largest
 * magnitude, the lowest column winning ties.  mask[n][k] in {0,1}.  K % m_group must be 0.
 * ------------------------------------------------------------------------------------------- */
void sbn_oracle_nm_mask(const float *W, int64_t N, int64_t K, int n_keep, int m_group,
                        uint8_t *mask)
{
    const int64_t G = K / m_group;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < G; ++g) {
            const float *w = W + n * K + g * m_group;
            uint8_t *m = mask + n * K + g * m_group;
            for (int j = 0; j < m_group; ++j) m[j] = 0;
            for (int r = 0; r < n_keep; ++r) {
                int best = -1;
                float best_a = -1.0f;
                for (int j = 0; j < m_group; ++j) {
                    if (m[j]) continue;
                    float a = fabsf(w[j]);
                    if (a > best_a) { best_a = a; best = j; }   /* strict: lower index wins ties */
                }
                m[best] = 1;
            }
        }
    }
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 1 (ternarise): W_q = clamp(round(W / scale), -1, +1); one fp32 division, half-to-even.
 * ------------------------------------------------------------------------------------------- */
void sbn_oracle_ternarize(const float *W, int64_t N, int64_t K, float scale, int8_t *q)
{
    const int64_t D = N * K;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < D; ++i) {
        volatile float v = W[i] / scale;
        float r = rintf(v);
        if (r > 1.0f) r = 1.0f;
        if (r < -1.0f) r = -1.0f;
        q[i] = (int8_t)r;
    }
}

/* Eq. 3: W_eff = W_q (.) M. */
void sbn_oracle_apply_mask(const int8_t *q, const uint8_t *mask, int64_t N, int64_t K, int8_t *weff)
{
    const int64_t D = N * K;
    for (int64_t i = 0; i < D; ++i) weff[i] = mask[i] ? q[i] : (int8_t)0;
}

/* ---------------------------------------------------------------------------------------------
 * Compressed 2:4 layout (see the header).  Requires a mask with exactly two ones per group of 4.
 * Returns 0 on success, -1 if some group does not hold exactly two kept positions.
 * ------------------------------------------------------------------------------------------- */
int sbn_oracle_pack24(const int8_t *q, const uint8_t *mask, int64_t N, int64_t K,
                      int8_t *vals, uint8_t *meta)
{
    const int64_t G = K / 4;
    if (K % 8 != 0) return -1;
    memset(meta, 0, (size_t)(N * (K / 8)));
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < G; ++g) {
            int idx[2], c = 0;
            for (int j = 0; j < 4; ++j)
                if (mask[n * K + 4 * g + j]) { if (c < 2) idx[c] = j; ++c; }
            if (c != 2) return -1;
            vals[n * (K / 2) + 2 * g]     = q[n * K + 4 * g + idx[0]];
            vals[n * (K / 2) + 2 * g + 1] = q[n * K + 4 * g + idx[1]];
            uint8_t nib = (uint8_t)(idx[0] | (idx[1] << 2));
            meta[n * (K / 8) + g / 2] |= (uint8_t)((g & 1) ? (nib << 4) : nib);
        }
    }
    return 0;
}

/* Inverse of the layout: rebuild W_eff [N][K] and the mask from vals/meta (used by route (ii)
 * checks and by the flip count). */
void sbn_oracle_unpack24(const int8_t *vals, const uint8_t *meta, int64_t N, int64_t K,
                         int8_t *weff, uint8_t *mask)
{
    const int64_t G = K / 4;
    if (weff) memset(weff, 0, (size_t)(N * K));
    if (mask) memset(mask, 0, (size_t)(N * K));
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < G; ++g) {
            uint8_t byte = meta[n * (K / 8) + g / 2];
            uint8_t nib = (g & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 15);
            int i0 = nib & 3, i1 = (nib >> 2) & 3;
            if (weff) {
                weff[n * K + 4 * g + i0] = vals[n * (K / 2) + 2 * g];
                weff[n * K + 4 * g + i1] = vals[n * (K / 2) + 2 * g + 1];
            }
            if (mask) {
                mask[n * K + 4 * g + i0] = 1;
                mask[n * K + 4 * g + i1] = 1;
            }
        }
    }
}

/* ---------------------------------------------------------------------------------------------
 * Packed storage of the kept values (not in the paper: a storage format of this build for the
 * weight-bound few-token regime).  A kept value is ternary: two bits hold t = v + 1 in {0, 1, 2}.
 * The two values of a group share a nibble, t0 | t1 << 2; group 2b sits in the low nibble of byte b
 * of its row, group 2b+1 in the high one.  vals2: [N][K/8] bytes -- with the metadata (unchanged,
 * [N][K/8] bytes) that is 2 bits per weight instead of 5.
 * Returns 0, or -1 on a non-ternary value (pack) / the unused field value 3 (unpack).
 * ------------------------------------------------------------------------------------------- */
int sbn_oracle_pack_vals2(const int8_t *vals, int64_t N, int64_t K, uint8_t *vals2)
{
    if (K % 8 != 0) return -1;
    memset(vals2, 0, (size_t)(N * (K / 8)));
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < K / 4; ++g) {
            int v0 = vals[n * (K / 2) + 2 * g], v1 = vals[n * (K / 2) + 2 * g + 1];
            if (v0 < -1 || v0 > 1 || v1 < -1 || v1 > 1) return -1;
            uint8_t nib = (uint8_t)((v0 + 1) | ((v1 + 1) << 2));
            vals2[n * (K / 8) + g / 2] |= (uint8_t)((g & 1) ? (nib << 4) : nib);
        }
    }
    return 0;
}

int sbn_oracle_unpack_vals2(const uint8_t *vals2, int64_t N, int64_t K, int8_t *vals)
{
    if (K % 8 != 0) return -1;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < K / 4; ++g) {
            uint8_t byte = vals2[n * (K / 8) + g / 2];
            int nib = (g & 1) ? (byte >> 4) : (byte & 15);
            int t0 = nib & 3, t1 = (nib >> 2) & 3;
            if (t0 == 3 || t1 == 3) return -1;
            vals[n * (K / 2) + 2 * g] = (int8_t)(t0 - 1);
            vals[n * (K / 2) + 2 * g + 1] = (int8_t)(t1 - 1);
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Part 1 of the path as one call: Eq. 1 scale on the dense W, Eq. 2 mask on |W|, Eq. 1 ternarise,
 * Eq. 3 mask application, then the compressed layout -- in exactly that order.
 * dense_q (optional) receives the unmasked W_q; mask_out (optional) the 0/1 mask.
 * ------------------------------------------------------------------------------------------- */
int sbn_oracle_quantize_mask_pack(const float *W, int64_t N, int64_t K,
                                  int8_t *vals, uint8_t *meta, float *scale_out,
                                  int8_t *dense_q, uint8_t *mask_out, int *near_tie)
{
    float gamma, scale;
    sbn_oracle_absmean_scale(W, N, K, &gamma, &scale, near_tie);
    uint8_t *mask = mask_out ? mask_out : (uint8_t *)malloc((size_t)(N * K));
    int8_t *q = dense_q ? dense_q : (int8_t *)malloc((size_t)(N * K));
    sbn_oracle_nm_mask(W, N, K, 2, 4, mask);
    sbn_oracle_ternarize(W, N, K, scale, q);
    int rc = sbn_oracle_pack24(q, mask, N, K, vals, meta);
    if (!mask_out) free(mask);
    if (!dense_q) free(q);
    if (scale_out) *scale_out = scale;
    return rc;
}

/* ---------------------------------------------------------------------------------------------
 * Activation quantiser (Sec. 2.1 and Algorithm 2's forward): per token t
 *   a = max_k |x|,  d = max(a, 1e-5),  s_x = 127 / d,
 *   x~ = clamp(round(x * s_x), -128, 127),  a_scale[t] = d / 127.
 * x is bf16, given as raw 16-bit patterns; widening to fp32 is exact.
 * ------------------------------------------------------------------------------------------- */
static inline float bf16_bits_to_f32(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

void sbn_oracle_quant_act(const uint16_t *x_bf16, int64_t T, int64_t K,
                          int8_t *xq, float *a_scale)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *x = x_bf16 + t * K;
        float a = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            float v = fabsf(bf16_bits_to_f32(x[k]));
            if (v > a) a = v;
        }
        float d = (a > SBN_ORACLE_EPS) ? a : SBN_ORACLE_EPS;
        volatile float s_x = 127.0f / d;
        for (int64_t k = 0; k < K; ++k) {
            volatile float p = bf16_bits_to_f32(x[k]) * s_x;
            float r = rintf(p);
            if (r > 127.0f) r = 127.0f;
            if (r < -128.0f) r = -128.0f;
            xq[t * K + k] = (int8_t)r;
        }
        volatile float as = d / 127.0f;
        a_scale[t] = as;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Algorithm 1, forward step  x~ = Q_a(Norm(x)).  The paper does not say which norm; it is read as
 * RMSNorm with a learned per-channel gain g (the norm BitNet-style blocks put in front of every
 * quantised linear layer):
 *     ms = mean_k x[k]^2            (double accumulation, one cast to float)
 *     r  = 1 / sqrt(ms + eps)       (float)
 *     xn[k] = (x[k] * r) * g[k]     (float, two rounded products; g == NULL means g = 1)
 * followed by Q_a of Sec. 2.1 on the float xn (no rounding to bf16 in between: the two steps are
 * one operation here).  near_tie[t] (optional) is set when a pairwise summation of the squares
 * gives a different float ms for row t; xn_out (optional) receives the normalised row.
 * ------------------------------------------------------------------------------------------- */
static double pairwise_sq_sum(const uint16_t *x, int64_t n)
{
    if (n <= 64) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double v = (double)bf16_bits_to_f32(x[i]);
            s += v * v;
        }
        return s;
    }
    int64_t h = n / 2;
    return pairwise_sq_sum(x, h) + pairwise_sq_sum(x + h, n - h);
}

void sbn_oracle_norm_quant_act(const uint16_t *x_bf16, int64_t T, int64_t K, const float *g,
                               float eps, int8_t *xq, float *a_scale, float *xn_out,
                               uint8_t *near_tie)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *x = x_bf16 + t * K;
        double S = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double v = (double)bf16_bits_to_f32(x[k]);
            S += v * v;
        }
        float ms = (float)(S / (double)K);
        if (near_tie) near_tie[t] = ((float)(pairwise_sq_sum(x, K) / (double)K) != ms);
        volatile float den = ms + eps;
        volatile float root = sqrtf(den);
        volatile float r = 1.0f / root;
        float *xn = (float *)malloc((size_t)K * sizeof(float));
        float a = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            volatile float p1 = bf16_bits_to_f32(x[k]) * r;
            volatile float p2 = g ? p1 * g[k] : p1;
            xn[k] = p2;
            float v = fabsf(p2);
            if (v > a) a = v;
        }
        float d = (a > SBN_ORACLE_EPS) ? a : SBN_ORACLE_EPS;
        volatile float s_x = 127.0f / d;
        for (int64_t k = 0; k < K; ++k) {
            volatile float p = xn[k] * s_x;
            float q = rintf(p);
            if (q > 127.0f) q = 127.0f;
            if (q < -128.0f) q = -128.0f;
            xq[t * K + k] = (int8_t)q;
            if (xn_out) xn_out[t * K + k] = xn[k];
        }
        volatile float as = d / 127.0f;
        a_scale[t] = as;
        free(xn);
    }
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 4, integer part, route (i): acc[t][n] = sum_k x~[t][k] * Wmat[n][k] with Wmat a plain
 * dense [N][K] int8 matrix (W_eff for the sparse layer, W_q for the dense BitLinear baseline).
 * ------------------------------------------------------------------------------------------- */
void sbn_oracle_acc_dense(const int8_t *xq, const int8_t *Wmat, int64_t T, int64_t N, int64_t K,
                          int32_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t s = 0;
            const int8_t *xr = xq + t * K;
            const int8_t *wr = Wmat + n * K;
            for (int64_t k = 0; k < K; ++k) s += (int32_t)xr[k] * (int32_t)wr[k];
            acc[t * N + n] = s;
        }
    }
}

/* Eq. 4, integer part, route (ii): the same sum taken from the compressed layout -- only the two
 * kept columns of every group contribute. */
void sbn_oracle_acc_packed(const int8_t *xq, const int8_t *vals, const uint8_t *meta,
                           int64_t T, int64_t N, int64_t K, int32_t *acc)
{
    const int64_t G = K / 4;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t s = 0;
            const int8_t *xr = xq + t * K;
            for (int64_t g = 0; g < G; ++g) {
                uint8_t byte = meta[n * (K / 8) + g / 2];
                uint8_t nib = (g & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 15);
                int i0 = nib & 3, i1 = (nib >> 2) & 3;
                s += (int32_t)xr[4 * g + i0] * (int32_t)vals[n * (K / 2) + 2 * g];
                s += (int32_t)xr[4 * g + i1] * (int32_t)vals[n * (K / 2) + 2 * g + 1];
            }
            acc[t * N + n] = s;
        }
    }
}

/* Route (ii) for a list of sampled outputs (t_idx[i], n_idx[i]); used on full-size shapes. */
void sbn_oracle_acc_packed_sampled(const int8_t *xq, const int8_t *vals, const uint8_t *meta,
                                   int64_t N, int64_t K, const int64_t *t_idx,
                                   const int64_t *n_idx, int64_t count, int32_t *acc)
{
    const int64_t G = K / 4;
    (void)N;
    for (int64_t i = 0; i < count; ++i) {
        int64_t t = t_idx[i], n = n_idx[i];
        int32_t s = 0;
        for (int64_t g = 0; g < G; ++g) {
            uint8_t byte = meta[n * (K / 8) + g / 2];
            uint8_t nib = (g & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 15);
            int i0 = nib & 3, i1 = (nib >> 2) & 3;
            s += (int32_t)xq[t * K + 4 * g + i0] * (int32_t)vals[n * (K / 2) + 2 * g];
            s += (int32_t)xq[t * K + 4 * g + i1] * (int32_t)vals[n * (K / 2) + 2 * g + 1];
        }
        acc[i] = s;
    }
}

/* Dense sum for a list of sampled outputs. */
void sbn_oracle_acc_dense_sampled(const int8_t *xq, const int8_t *Wmat, int64_t N, int64_t K,
                                  const int64_t *t_idx, const int64_t *n_idx, int64_t count,
                                  int32_t *acc)
{
    (void)N;
    for (int64_t i = 0; i < count; ++i) {
        int64_t t = t_idx[i], n = n_idx[i];
        int32_t s = 0;
        for (int64_t k = 0; k < K; ++k) s += (int32_t)xq[t * K + k] * (int32_t)Wmat[n * K + k];
        acc[i] = s;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 4, scaling: y[t][n] = float(acc) * (scale * a_scale[t]) (+ bias[n]); s "absorbs the
 * quantisation scales".  Two fp32 multiplications in this association, then the optional add.
 * ------------------------------------------------------------------------------------------- */
void sbn_oracle_dequant(const int32_t *acc, float scale, const float *a_scale, const float *bias,
                        int64_t T, int64_t N, float *y)
{
    for (int64_t t = 0; t < T; ++t) {
        volatile float s = scale * a_scale[t];
        for (int64_t n = 0; n < N; ++n) {
            volatile float v = (float)acc[t * N + n] * s;
            if (bias) v = v + bias[n];
            y[t * N + n] = v;
        }
    }
}

/* fp32 -> bf16 bit pattern, round-to-nearest-even (finite inputs). */
void sbn_oracle_f32_to_bf16(const float *y, int64_t count, uint16_t *out)
{
    for (int64_t i = 0; i < count; ++i) {
        uint32_t u;
        memcpy(&u, &y[i], 4);
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7FFFu + lsb;
        out[i] = (uint16_t)(u >> 16);
    }
}

/* ---------------------------------------------------------------------------------------------
 * Flip-rate numerator (Sec. 4): || m(w_t) - m(w_{t-1}) ||_1, the number of positions whose mask
 * bit differs; both masks given as 0/1 [N][K] arrays.  r_t = count / (N*K).
 * ------------------------------------------------------------------------------------------- */
uint64_t sbn_oracle_flip_count(const uint8_t *mask_a, const uint8_t *mask_b, int64_t N, int64_t K)
{
    uint64_t c = 0;
    const int64_t D = N * K;
    for (int64_t i = 0; i < D; ++i) c += (uint64_t)((mask_a[i] != 0) != (mask_b[i] != 0));
    return c;
}

int sbn_oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
