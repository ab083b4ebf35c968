/*
 * sbn.h -- C ABI of libsbn: the 2:4-sparse ternary BitLinear layer of Sparse-BitNet on one
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the forward hot path of the Sparse-BitLinear layer (Sec. 2.2, Eq. 2-4,
 * Algorithm 2) and of the dense BitLinear it is compared with (Sec. 2.1, Eq. 1):
 *
 *   part 1  sbn_quantize_mask_pack   W (fp32 master weights) -> ternary W_q (Eq. 1), 2:4 mask from
 *                                    |W| of the pre-quantised weights (Eq. 2), W_eff = W_q (.) M
 *                                    (Eq. 3), stored as compressed values + 2-bit index metadata
 *   part 2  sbn_quant_act            x (bf16) -> per-token absmax int8 x~ and its scale (Sec. 2.1)
 *   part 3  sbn_sparse_bitlinear     y = s * (W_eff x~) (Eq. 4): sparse int8 tensor-core GEMM,
 *                                    int32 accumulation, scales applied in the epilogue
 *   base    sbn_bitlinear            y = gamma * matmul(W_q, x~) (Sec. 2.1), dense int8 GEMM
 *
 * Notation: T = tokens, K = d_in, N = d_out.  All matrices are row-major.
 *
 * General rules
 *   - Every pointer marked "device" is a CUDA device pointer owned by the caller.  The library
 *     never allocates or frees device memory and keeps no reference after the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *     work on it; nothing here synchronises except sbn_check_status.
 *   - Errors are return codes.  Argument errors are detected on the host before anything is
 *     launched.  Device-side waits are bounded; a wait that runs out records SBN_ERR_TIMEOUT in a
 *     device status word that sbn_check_status reads back.
 *   - The kernels are launched with programmatic stream serialisation: a kernel's set-up may
 *     overlap the end of the kernel before it on the same stream, results are those of plain
 *     stream order.  One rule follows for callers that write vals / meta / dense_q with a kernel
 *     of their own: that kernel must not signal programmatic launch completion early
 *     (cudaTriggerProgrammaticLaunchCompletion / griddepcontrol.launch_dependents), because the
 *     few-token GEMM fetches weights before its dependency wait.  Copies and ordinary kernels are
 *     fine.  SBN_DISABLE_PDL=1 in the environment turns the overlap off.
 *   - Inputs must be finite.  NaN/Inf give unspecified results.
 *   - Shape limits of the GPU path: N % 128 == 0, K % 128 == 0, T >= 1, K <= 2^20, pointers
 *     16-byte aligned (cudaMalloc alignment is always enough).
 *
 * Compressed 2:4 layout (the paper leaves the layout to the kernel; this is the library's):
 *   groups are 4 consecutive columns of a row, aligned to column 0; group g of row n keeps the
 *   columns 4g+i0 < 4g+i1;
 *     vals[n][2g]   = W_q[n][4g+i0],  vals[n][2g+1] = W_q[n][4g+i1]          int8  [N][K/2]
 *     nibble(g)     = i0 | (i1 << 2)
 *     meta[n][b]    = nibble(2b) | (nibble(2b+1) << 4)                       uint8 [N][K/8]
 *
 * Storage order of the GEMM operands ("tiled"): vals, meta, dense_q and xq are NOT stored as the
 * plain row-major arrays above but tile by tile, each tile being the exact shared-memory image
 * the tensor-core instruction consumes, so that a tile is one contiguous block of HBM.  Every
 * buffer has the same number of bytes as its row-major form (xq: tokens padded to a multiple of
 * 16) and is a pure permutation of it.  With KB = K/128, r = n % 128 (or t % 8 for xq), all
 * offsets in bytes:
 *     vals    element (n, c), c in [0, K/2):   ((n/128)*KB + c/64)*8192 + r*64
 *                                              + ((((c%64)/16) ^ ((r/2)%4)) * 16) + c%16
 *     meta    element (n, b), b in [0, K/8):   ((n/128)*KB + b/16)*2048 + r*16 + b%16
 *     dense_q element (n, k), k in [0, K):     ((n/128)*KB + k/128)*16384 + (r/8)*1024 + (r%8)*128
 *                                              + ((((k%128)/16) ^ (r%8)) * 16) + k%16
 *     xq      element (t, k):                  ((k/128)*TB8 + t/8)*1024 + (t%8)*128
 *                                              + ((((k%128)/16) ^ (t%8)) * 16) + k%16,
 *             TB8 = 2*ceil(T/16); buffer size sbn_xq_bytes(T, K) = TB8 * KB * 1024
 */
#ifndef SBN_H_
#define SBN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SBN_OK = 0,
    SBN_ERR_NULL = 1,        /* a required pointer is NULL */
    SBN_ERR_SHAPE = 2,       /* a dimension is <= 0 or breaks the divisibility rules above */
    SBN_ERR_ALIGN = 3,       /* a pointer is not 16-byte aligned */
    SBN_ERR_UNSUPPORTED = 4, /* pattern other than 2:4 / 6:8, unknown dtype or op */
    SBN_ERR_WORKSPACE = 5,   /* workspace missing or smaller than sbn_workspace_bytes() */
    SBN_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed (launch, tensor map, ...) */
    SBN_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (see sbn_check_status) */
    SBN_ERR_TOO_LARGE = 8    /* problem exceeds what the library's built-in scratch can serve */
} sbn_status;

typedef enum { SBN_OUT_F32 = 0, SBN_OUT_BF16 = 1 } sbn_out_dtype;

typedef enum {
    SBN_OP_QUANTIZE_MASK_PACK = 0,
    SBN_OP_QUANT_ACT = 1,
    SBN_OP_SPARSE_BITLINEAR = 2,
    SBN_OP_BITLINEAR = 3,
    SBN_OP_BACKWARD = 4
} sbn_op;

/* Host, pure.  Bytes of the tiled int8 activation buffer xq for T tokens of K columns. */
size_t sbn_xq_bytes(int T, int K);

/* Host, pure.  Bytes of device workspace the given call needs for these sizes (0 if none).
 * T is ignored by SBN_OP_QUANTIZE_MASK_PACK. */
size_t sbn_workspace_bytes(int op, int T, int N, int K);

/*
 * Part 1 -- Eq. 1 (absmean ternary quantiser), Eq. 2 (magnitude N:M mask from the master
 * weights), Eq. 3 (W_eff = W_q (.) M), in that order, then the compressed layout above.
 *   gamma  = sum|W| / (N*K), accumulated in fp64, rounded to fp32 once, over the whole dense W
 *   scale  = max(gamma, 1e-5)                            (Algorithm 2's clamp)
 *   W_q    = clamp(round_half_even(W / scale), -1, +1)   (fp32 division)
 *   mask   = the two largest |W| of every group of four; equal magnitudes -> lower column kept
 * Arguments
 *   W          device, fp32 [N][K], read only
 *   n_keep, m_group  the N:M pattern: 2:4, or 6:8 (see "The 6:8 pattern" below); anything else
 *              SBN_ERR_UNSUPPORTED
 *   vals       device out, int8, N*K/2 bytes, tiled order
 *   meta       device out, uint8, N*K/8 bytes, tiled order; may be the same buffer as prev_meta
 *   w_scale    device out, one fp32: `scale`
 *   dense_q    device out or NULL, int8, N*K bytes, tiled order: the unmasked W_q (operand of
 *              sbn_bitlinear)
 *   prev_meta  device or NULL, uint8, N*K/8 bytes, tiled order: metadata of the previous step's mask
 *   flip_bits  device out or NULL (required iff prev_meta != NULL), one uint64: number of
 *              positions whose mask bit differs from prev_meta's, i.e. the numerator of the flip
 *              rate r_t = ||m(w_t) - m(w_{t-1})||_1 / D (Sec. 4); overwritten, not accumulated
 *   ws         device workspace of sbn_workspace_bytes(SBN_OP_QUANTIZE_MASK_PACK, 0, N, K)
 *              bytes; contents need no initialisation; must not be shared by calls that may run
 *              concurrently.  It holds the per-CTA partial sums of |W| and a generation word that
 *              the kernel advances on every execution, so a call captured in a CUDA graph may be
 *              replayed on the same workspace (each replay tells its own partial sums from the
 *              previous replay's).  The 2:4 kernel also leaves the scale it found there, tagged with
 *              W and the shape: the next call for the same matrix on the same workspace starts from it
 *              (as if it were a job's gamma_hint: no sample of the matrix, almost nothing to fix up) --
 *              a speed-up for loops that re-pack the same buffers every step, never a change of the
 *              result; bytes that do not carry the tag are ignored
 * Residency rule (this call, the _bf16, _batched and _static_ws forms alike).  The kernel is one
 * persistent grid of at most one CTA per SM (1024 threads each) whose CTAs exchange their partial
 * sums through the workspace, so ALL of its CTAs must be resident at the same time.  On a GPU that
 * runs nothing else that is always so.  Two such calls that may overlap on the GPU (different
 * streams, no ordering between them) can each occupy part of the SMs and then wait for CTAs that
 * cannot start; neither hangs -- every wait is bounded -- but both can end with SBN_ERR_TIMEOUT
 * from sbn_check_status and unfinished outputs.  Order such calls (one stream, or events), or
 * give all matrices to one sbn_quantize_mask_pack_batched call.  The same holds next to any other
 * kernel that keeps SMs fully occupied for seconds.
 */
sbn_status sbn_quantize_mask_pack(const float *W, int N, int K, int n_keep, int m_group,
                                  int8_t *vals, uint8_t *meta, float *w_scale, int8_t *dense_q,
                                  const uint8_t *prev_meta, unsigned long long *flip_bits,
                                  void *ws, size_t ws_bytes, void *stream);

/*
 * The 6:8 pattern (Sec. 2.2 with N:M = 6:8, the pattern of the paper's main results and of its
 * throughput table): of every 8 consecutive input weights the 6 largest |W| are kept (equal
 * magnitudes -> lower column kept); gamma, scale and W_q as above, from the dense matrix.
 * The paper does not say how 6:8 reaches 2:4 hardware.  Here a group of 8 columns is covered by
 * three overlapping 4-column windows (columns 0-3, 2-5, 4-7); the 6 kept columns are dealt out so
 * that each window holds exactly two of them, which makes the [N][K] 6:8 matrix a 2:4 matrix
 * [N][K'] with K' = sbn_expanded_k(K, 6, 8) = 3K/2 over activations expanded the same way
 * (K' column 12 g + 4 w + s holds column 8 g + 2 w + s; sbn_quant_act_expand68 writes them).
 * sbn_sparse_bitlinear then runs unchanged with K' in place of K: 3/4 of the dense MMA work.
 * With n_keep = 6, m_group = 8, sbn_quantize_mask_pack and sbn_quantize_mask_pack_bf16 take
 *   K          a multiple of 256 (else SBN_ERR_SHAPE)
 *   vals       N*K'/2 bytes and meta N*K'/8 bytes: the 2:4 form of the [N][K'] matrix, tiled order
 *   prev_meta  N*K'/8 bytes, the same form; flip_bits counts differing bits of the 6:8 masks [N][K]
 *   dense_q    must be NULL (the dense W_q does not depend on the pattern; SBN_ERR_UNSUPPORTED)
 * Which window carries a kept column is this library's choice (window 0 takes the kept ones of
 * columns 0,1 and fills up with the lowest kept of 2,3; window 2 takes the kept ones of 6,7 and
 * fills up with the highest kept of 4,5; window 1 takes the rest); W_eff and the mask are unique.
 */
int sbn_expanded_k(int K, int n_keep, int m_group);   /* K for 2:4, 3K/2 for 6:8 (K % 256 == 0), else 0 */

/*
 * The same operation on bf16 master weights (Sec. 2.2 keeps the master weight "e.g. in bf16"): W is
 * read as bf16 [N][K] (16-byte aligned), every value is taken as the real number it represents, and
 * everything else -- arguments, results, exactness -- is as above.  Half the weight traffic.
 */
sbn_status sbn_quantize_mask_pack_bf16(const void *W_bf16, int N, int K, int n_keep, int m_group,
                                       int8_t *vals, uint8_t *meta, float *w_scale, int8_t *dense_q,
                                       const uint8_t *prev_meta, unsigned long long *flip_bits,
                                       void *ws, size_t ws_bytes, void *stream);

/*
 * Part 1 for many matrices in ONE launch -- the dynamic-mask training step recomputes the mask of
 * every BitLinear at every step (Sec. 2.3, "Dynamic Mask Recomputation"; Algorithm 1).  Each job
 * is exactly one sbn_quantize_mask_pack call (same arguments, same results, bit for bit); the
 * kernel streams through the matrices without a pause between them: the exchange of partial sums,
 * the threshold and the fix-up of one matrix run under the pass over the next ones.
 *   jobs   host array of `count` jobs; fully read before the call returns (pageable memory is
 *          fine: the jobs travel to the device as kernel arguments, 48 per small launch, not through
 *          a staging copy, so the call only enqueues and never blocks on the stream)
 *   ws     device workspace of sbn_batch_workspace_bytes(count) bytes; no initialisation needed;
 *          not to be shared by calls that may run concurrently
 */
typedef struct {
    const void *W;                    /* device, [N][K], fp32 or (w_bf16 != 0) bf16 */
    int N, K;
    int8_t *vals;                     /* device out, tiled */
    uint8_t *meta;                    /* device out, tiled; may equal prev_meta */
    float *w_scale;                   /* device out, one fp32 */
    int8_t *dense_q;                  /* device out or NULL */
    const uint8_t *prev_meta;         /* device or NULL */
    unsigned long long *flip_bits;    /* device out; required iff prev_meta != NULL */
    int w_bf16;                       /* 0: W is fp32; 1: W is bf16 (see sbn_quantize_mask_pack_bf16) */
    const float *gamma_hint;          /* device, one fp32, or NULL: an estimate of this matrix's gamma, e.g. the
                                         w_scale of the previous training step (may be the very w_scale buffer
                                         above: it is read before it is written).  A speed hint only -- results
                                         never depend on it.  With a hint within 0.5 % of gamma the kernel need
                                         not sample the matrix first and finds almost nothing to fix up afterwards; a
                                         hint that is further off costs a second pass over that matrix, one that is
                                         not a positive finite number is ignored */
} sbn_pack_job;
size_t sbn_batch_workspace_bytes(int count);
sbn_status sbn_quantize_mask_pack_batched(int count, const sbn_pack_job *jobs, void *ws, size_t ws_bytes,
                                          void *stream);

/*
 * Same operation as sbn_quantize_mask_pack, for callers that have no workspace to give.
 * (The paper has no counterpart to this call; it exists for integration reasons only.)
 *
 * Some hosts of this library cannot obtain device memory at the point where they call it: a
 * framework that reserved nearly all of the GPU for its own pool at start-up (cudaMalloc then
 * fails, and the pool cannot be asked from plain C), a plug-in whose "enqueue" hook is forbidden
 * to allocate, or a latency-critical loop that must avoid cudaMalloc because it synchronises the
 * whole device.  For them the scratch of the two-pass quantiser (the per-CTA partial sums of
 * |W|) lives in a fixed array inside the library image: SBN_STATIC_SCRATCH_BYTES bytes of
 * device memory that every GPU which loads the library keeps until the process exits.
 *
 * Arguments are those of sbn_quantize_mask_pack without ws/ws_bytes; inputs and outputs are
 * still the caller's buffers, and the results are bit-identical to that call's.
 * Limits and rules
 *   - 2:4 only: n_keep = 2, m_group = 4; the 6:8 pattern returns SBN_ERR_UNSUPPORTED here.
 *   - N*K must not exceed SBN_STATIC_MAX_ELEMS, and the scratch the shape needs must fit in
 *     SBN_STATIC_SCRATCH_BYTES; otherwise SBN_ERR_TOO_LARGE is returned and nothing is launched.
 *   - The call itself never allocates or frees memory (no cudaMalloc/cudaFree, no allocating
 *     library routine).
 *   - The first call on each device looks up the device address of the built-in array (once per
 *     device, with that device current).  If nothing of this library has run on the device yet,
 *     that lookup is also when the CUDA runtime loads the library's device code, which reserves
 *     memory for the image (the built-in array included): it is the calls after the first that
 *     are allocation-free.  Make that first call before starting any stream capture on the
 *     device.
 *   - All calls on one device share the one array, and it keeps whatever the last call left in
 *     it (each call overwrites every slot it later reads, so nothing needs clearing).  Two such
 *     calls that may overlap on the GPU -- different streams, no ordering between them -- race
 *     on it and give wrong scales; order them, or use sbn_quantize_mask_pack with separate
 *     workspaces.
 */
#define SBN_STATIC_SCRATCH_BYTES 8192
#define SBN_STATIC_MAX_ELEMS (1ll << 28)
sbn_status sbn_quantize_mask_pack_static_ws(const float *W, int N, int K, int n_keep, int m_group,
                                            int8_t *vals, uint8_t *meta, float *w_scale,
                                            int8_t *dense_q, const uint8_t *prev_meta,
                                            unsigned long long *flip_bits, void *stream);

/*
 * Part 2 -- per-token absmax int8 activation quantiser (Sec. 2.1; Algorithm 2, forward step 1):
 *   a = max_k |x[t][k]|, d = max(a, 1e-5), s_x = 127 / d,
 *   xq[t][k] = clamp(round_half_even(x[t][k] * s_x), -128, 127),  a_scale[t] = d / 127.
 *   x_bf16   device, bf16 [T][K]
 *   xq       device out, int8, sbn_xq_bytes(T, K) bytes, tiled order (see above)
 *   a_scale  device out, fp32 [T]
 */
sbn_status sbn_quant_act(const void *x_bf16, int T, int K, int8_t *xq, float *a_scale,
                         void *stream);

/*
 * The same quantiser writing the activations expanded for the 6:8 pattern (see above): the codes
 * and a_scale are exactly those of sbn_quant_act; xq is the tiled form of the [T][K'] matrix with
 * K' = 3K/2, xq'[t][12 g + 4 w + s] = xq[t][8 g + 2 w + s] (g < K/8, w < 3, s < 4).
 *   K    a multiple of 256
 *   xq   device out, sbn_xq_bytes(T, 3K/2) bytes
 */
sbn_status sbn_quant_act_expand68(const void *x_bf16, int T, int K, int8_t *xq, float *a_scale,
                                  void *stream);

/*
 * Part 2 with the preceding normalisation fused in -- Algorithm 1, forward: x~ = Q_a(Norm(x)).
 * The paper does not name the norm; it is taken as RMSNorm with a per-channel gain:
 *   ms = mean_k x[t][k]^2 (accumulated in fp64),  r = 1 / sqrt(ms + eps),
 *   xn[k] = (x[t][k] * r) * gain[k]              (fp32; gain == NULL means all ones)
 * followed by the quantiser above applied to the fp32 xn (which is never written to memory).
 *   x_bf16   device, bf16 [T][K], K % 128 == 0, K <= 16384 (else SBN_ERR_UNSUPPORTED)
 *   gain     device, fp32 [K], 16-byte aligned, or NULL
 *   eps      >= 0
 *   xq, a_scale   as for sbn_quant_act
 * Asynchronous on `stream`; caller owns all buffers.
 */
sbn_status sbn_norm_quant_act(const void *x_bf16, int T, int K, const float *gain, float eps,
                              int8_t *xq, float *a_scale, void *stream);

/* The same with the codes written expanded for the 6:8 pattern (as sbn_quant_act_expand68:
 * K % 256 == 0, xq of sbn_xq_bytes(T, 3K/2) bytes). */
sbn_status sbn_norm_quant_act_expand68(const void *x_bf16, int T, int K, const float *gain,
                                       float eps, int8_t *xq, float *a_scale, void *stream);

/*
 * Part 3 -- Eq. 4: acc[t][n] = sum_k xq[t][k] * W_eff[n][k] in int32 (exact), then
 *   y[t][n] = float(acc[t][n]) * (w_scale * a_scale[t]) (+ bias[n]),
 * written as fp32 or as bf16 (round-to-nearest-even of the fp32 value).
 *   xq, a_scale   device, outputs of sbn_quant_act
 *   vals, meta, w_scale  device, outputs of sbn_quantize_mask_pack (w_scale stays on the device)
 *   bias          device fp32 [N] or NULL
 *   y             device out, [T][N] of `dt`
 *   acc_out       device out or NULL, int32 [T][N]: the raw accumulators (for parity checks)
 *   ws, ws_bytes  device workspace of sbn_workspace_bytes(SBN_OP_SPARSE_BITLINEAR, T, N, K)
 *                 bytes (may be NULL when that is 0).  It must be zero-filled before its first
 *                 use; every call that completes leaves it zero-filled again (split-K sums for
 *                 small T live there), so it can be reused without clearing
 */
sbn_status sbn_sparse_bitlinear(const int8_t *xq, const float *a_scale, int T,
                                const int8_t *vals, const uint8_t *meta, const float *w_scale,
                                int N, int K, const float *bias, void *y, sbn_out_dtype dt,
                                int32_t *acc_out, void *ws, size_t ws_bytes, void *stream);

/*
 * Parts 2 and 3 in one kernel, for few tokens -- Algorithm 2's forward as it stands: the per-token
 * absmax quantiser (Sec. 2.1) and Eq. 4.  Results are those of sbn_quant_act followed by
 * sbn_sparse_bitlinear (resp. sbn_bitlinear), bit for bit; what is saved is a kernel launch.  That
 * pays when launches are plainly serialised (measured 9.8 us against 12.8 us per layer at T = 8);
 * in a stream of this library's own calls, which overlap through programmatic dependent launch,
 * the two separate calls are faster (6.4 us against 7.6 us).  The quantised activations never reach
 * memory.
 *   x_bf16        device, bf16 [T][K], 16-byte aligned, K % 128 == 0
 *   a_scale_out   device out or NULL, fp32 [T]: the per-token scales d / 127
 *   the other arguments as for sbn_sparse_bitlinear / sbn_bitlinear; no workspace
 * Few tokens only: T <= 256 and K >= 256, else SBN_ERR_UNSUPPORTED (meant for T <= 32; beyond that
 * every 32-token tile quantises its own tokens again for each of the N / 128 row tiles).
 */
sbn_status sbn_quant_act_sparse_bitlinear(const void *x_bf16, int T, const int8_t *vals,
                                          const uint8_t *meta, const float *w_scale, int N, int K,
                                          const float *bias, void *y, sbn_out_dtype dt,
                                          int32_t *acc_out, float *a_scale_out, void *stream);
sbn_status sbn_quant_act_bitlinear(const void *x_bf16, int T, const int8_t *dense_q,
                                   const float *w_scale, int N, int K, const float *bias, void *y,
                                   sbn_out_dtype dt, int32_t *acc_out, float *a_scale_out,
                                   void *stream);

/*
 * Packed weights for the weight-bound few-token regime (not in the paper: a storage format of this
 * library).  A kept value is ternary, so two bits hold it: t = v + 1 in {0, 1, 2}.  sbn_pack_vals2
 * turns the value bytes of the compressed form into nibbles, t0 | t1 << 2 per group, group 2b in the
 * low nibble of byte b of its row and group 2b+1 in the high one: vals2 is [N][K/8] bytes, stored
 * tile by tile exactly like meta (same offsets).  With the metadata, which stays as it is, a
 * weight costs 2 bits instead of 5.
 *   vals    device, output of sbn_quantize_mask_pack (2:4), tiled order
 *   vals2   device out, N*K/8 bytes, 16-byte aligned
 * sbn_sparse_bitlinear_packed is sbn_sparse_bitlinear on (vals2, meta): same results, bit for bit.
 * The kernel fetches 4 KB per 128 x 128 block instead of 10 KB and expands the values in shared
 * memory next to the MMAs.  Few tokens only: T <= 1024 and K >= 256, else SBN_ERR_UNSUPPORTED
 * (intended for T <= 32 on large matrices, where the weight stream is what a call costs); no
 * workspace.  Like every producer of weights, a caller's kernel that writes vals2 must not signal
 * programmatic launch completion early.
 */
sbn_status sbn_pack_vals2(const int8_t *vals, int N, int K, uint8_t *vals2, void *stream);
sbn_status sbn_sparse_bitlinear_packed(const int8_t *xq, const float *a_scale, int T,
                                       const uint8_t *vals2, const uint8_t *meta,
                                       const float *w_scale, int N, int K, const float *bias,
                                       void *y, sbn_out_dtype dt, int32_t *acc_out, void *stream);

/*
 * Baseline -- dense BitLinear (Sec. 2.1): same as above with the unmasked ternary
 * dense_q int8 [N][K] in place of vals/meta.
 */
sbn_status sbn_bitlinear(const int8_t *xq, const float *a_scale, int T,
                         const int8_t *dense_q, const float *w_scale,
                         int N, int K, const float *bias, void *y, sbn_out_dtype dt,
                         int32_t *acc_out, void *ws, size_t ws_bytes, void *stream);

/*
 * Backward of one Sparse-BitLinear layer under the dual straight-through estimator -- Sec. 2.3, Eq. 5
 * (the mask is transparent to the gradient, like the quantiser), Algorithm 1 "Backward", Algorithm 2's
 * backward (the weight function returns g_out unchanged).  With y = F.linear(x_q, w_masked), x_q the
 * fake-quantised activations xq[t][k] * a_scale[t] and w_masked = W_eff * w_scale:
 *   dW[n][k] = sum_t dY[t][n] * x_q[t][k]       DENSE: every master weight gets its gradient, pruned
 *                                               ones included (the mask is NOT applied)
 *   dX[t][k] = sum_n dY[t][n] * w_masked[n][k]  through the activation quantiser as the identity
 * Precision (the paper states none; its models train with bf16 tensors): dY is bf16, the saved operands
 * enter as a bf16 run holds them, x_q = bf16(xq * a_scale) and w_masked = W_eff * bf16(w_scale); products
 * are exact, sums are accumulated in fp32 on the tensor cores; dW leaves as fp32, dX as bf16.
 *   dY_bf16   device, bf16 [T][N]
 *   xq, a_scale           device, the forward's quantised activations (tiled) and scales; needed for dW
 *   vals, meta, w_scale   device, the forward's packed weights; needed for dX
 *   dX_bf16   device out, bf16 [T][K], or NULL to skip
 *   dW        device out, fp32 [N][K], or NULL to skip (overwritten, not accumulated)
 *   ws        device workspace of sbn_workspace_bytes(SBN_OP_BACKWARD, T, N, K) bytes, 256-byte aligned
 *             (W_eff^T [K][N] and x_q [T][K] in bf16); no initialisation needed
 * The bias gradient (a column sum of dY) is not computed here.
 */
sbn_status sbn_bitlinear_backward(const void *dY_bf16, int T, const int8_t *xq, const float *a_scale,
                                  const int8_t *vals, const uint8_t *meta, const float *w_scale,
                                  int N, int K, void *dX_bf16, float *dW, void *ws, size_t ws_bytes,
                                  void *stream);

/*
 * Whole forward of one layer from HOST activations (Algorithm 2's forward with pre-packed
 * weights): copies x (bf16 [T][K], host, ideally pinned) to `x_dev`, runs sbn_quant_act and
 * sbn_sparse_bitlinear (or sbn_bitlinear when vals == NULL and dense_q != NULL), and copies
 * y ([T][N] of `dt`) back to `y_host`.  All on `stream`; returns after enqueueing.
 *   x_dev   device staging, T*K*2 bytes;  xq_dev  device, sbn_xq_bytes(T, K);  a_scale_dev device, T*4
 *   y_dev   device staging for y
 * Weights (vals/meta or dense_q, w_scale, bias) are device pointers as above.
 */
sbn_status sbn_layer_forward_host(const void *x_bf16_host, int T, int K,
                                  void *x_dev, int8_t *xq_dev, float *a_scale_dev,
                                  const int8_t *vals, const uint8_t *meta, const int8_t *dense_q,
                                  const float *w_scale, int N, const float *bias,
                                  void *y_dev, void *y_host, sbn_out_dtype dt,
                                  void *ws, size_t ws_bytes, void *stream);

/*
 * The compressed weights between the library's tiled storage order and the plain row-major arrays
 * of the layout definition at the top of this file (Sec. 2.2 asks for "a well-defined N:M
 * metadata/layout"; vals [N][K/2] and meta [N][K/8] as defined there are that layout, the tiled order
 * is how this library keeps them in memory for its GEMM).  Pure permutations, device to device:
 *   sbn_unpack_canonical   tiled vals / meta (outputs of sbn_quantize_mask_pack) -> plain arrays, for
 *                          storing, inspecting or exporting packed weights
 *   sbn_tile_canonical     plain arrays -> tiled order, for loading packed weights produced elsewhere
 *                          (values must be -1, 0, +1 and every metadata nibble one of 4, 8, 9, 12, 13,
 *                          14 -- not checked)
 *   N, K       as for the pack call (for the 6:8 form pass K' = sbn_expanded_k(K, 6, 8))
 *   vals / meta pairs: either pair may be NULL (both pointers) to convert only the other one
 * Source and destination must be different buffers (SBN_ERR_UNSUPPORTED otherwise), 16-byte aligned.
 * Asynchronous on `stream`.  sbn_tile_canonical writes weights: like every weight producer it gives
 * the kernels behind it no early start.
 */
sbn_status sbn_unpack_canonical(const int8_t *vals, const uint8_t *meta, int N, int K,
                                int8_t *vals_out, uint8_t *meta_out, void *stream);
sbn_status sbn_tile_canonical(const int8_t *vals_plain, const uint8_t *meta_plain, int N, int K,
                              int8_t *vals, uint8_t *meta, void *stream);

/* Synchronises `stream`, returns SBN_ERR_TIMEOUT if any kernel since the last call gave up on a
 * bounded wait (and clears that record), SBN_ERR_CUDA if the stream reports an error, else
 * SBN_OK. */
sbn_status sbn_check_status(void *stream);

/* Static string for a status code. */
const char *sbn_status_string(sbn_status s);

/* Tuning/diagnostic knob (host state, not thread-safe).  token_tile: 0 = automatic; 64, 128 or
 * 256 = force the single-CTA kernel with that token-tile width; a negative value -BN = force the
 * CTA-pair kernel with BN tokens per tile (rounded to a multiple of 16, capped at 240 sparse /
 * 256 dense; with split_k = 1 its variant with one M-tile per CTA).  split_k: 0 = automatic; k > 0 = split K k ways through int32 atomics in the
 * workspace (single-CTA kernel); -2, -3, -4, -8 = split K inside thread-block clusters of that many
 * CTAs (token tile 64, or 32 / 128 if token_tile says so; no workspace; -2, -3, -4 also set the
 * cluster size of sbn_sparse_bitlinear_packed and of the sbn_quant_act_*bitlinear kernels).  Results do not depend on
 * it. */
void sbn_set_gemm_tuning(int token_tile, int split_k);

/* Diagnostic for tests of the failure path (host state, not thread-safe; acts on the current device).
 * wait_limit_us: limit of every bounded device-side wait from now on, in microseconds (0 = back to
 * the default of 2 s).  break_waits != 0: the GEMM kernels' load producers issue no loads and the last
 * CTA of the pack kernel does not publish its partial sum, so the waits of the other roles run out:
 * every role then leaves through the kernel's abort path, the kernel returns (nothing traps, nothing
 * waits without limit), outputs are unspecified and the next sbn_check_status reports
 * SBN_ERR_TIMEOUT.  sbn_set_wait_test(0, 0) restores normal operation. */
sbn_status sbn_set_wait_test(int break_waits, unsigned long long wait_limit_us);

/* Diagnostic for timing experiments on the large-T (CTA-pair) GEMM kernel: what its K-loop costs without
 * parts of itself.  RESULTS ARE WRONG while flags != 0 -- timing only; 0 restores normal operation.
 * Host state, not thread-safe.  Bits: 1 = operands stay resident in shared memory (loads only for the
 * first pipeline fill of a launch), 2 = never load weights and metadata, 4 = never load activations,
 * 8 = no metadata copies into tensor memory, 16 / 32 = issue every stage's MMAs twice / four times.
 * Used by `bench.py --workload mmaprobe`. */
void sbn_set_gemm_probe(int flags);

/* Diagnostic: what the dispatcher would run for this shape (host only, launches nothing).
 * out4[0] = kernel (0 single-CTA tiles, 1 cluster split-K, 2 CTA pair with 512-feature tiles, 3 CTA
 * pair with 256-feature tiles and double-buffered accumulators), out4[1] = tokens per tile,
 * out4[2] = split-K factor through global memory (1 = none), out4[3] = cluster size (0 = none).
 * All zero for an illegal shape. */
void sbn_plan_gemm(int sparse, int T, int N, int K, int *out4);

/* Number of kernels the library has launched since it was loaded (all calls, all streams). */
unsigned long long sbn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SBN_H_ */
