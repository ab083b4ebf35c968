"""CPU oracle for the 2:4-sparse ternary BitLinear path (Sparse-BitNet, Eq. 1-4, Algorithm 2).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The product (the CUDA library and its Python binding) never imports this
package, and this package never imports the product.

The arithmetic lives in ``sbn_oracle.c`` (plain C, one function per passage of the paper); this
module compiles it with gcc on first use and wraps every function for numpy arrays.  No value
that enters or leaves these functions ever comes from the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sbn_oracle.c")
_LIB = os.path.join(_HERE, "libsbn_oracle.so")
_lock = threading.Lock()
_lib = None

EPS = np.float32(1e-5)


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared library next to its source (gcc, OpenMP)."""
    with _lock:
        if (not force and os.path.exists(_LIB)
                and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
            return _LIB
        cmd = ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-std=c11", "-o", _LIB + ".tmp", _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(_LIB + ".tmp", _LIB)
        return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp, i32, f32 = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        sig = {
            "sbn_oracle_absmean_scale": (None, [vp, i64, i64, vp, vp, vp]),
            "sbn_oracle_nm_mask": (None, [vp, i64, i64, i32, i32, vp]),
            "sbn_oracle_ternarize": (None, [vp, i64, i64, f32, vp]),
            "sbn_oracle_apply_mask": (None, [vp, vp, i64, i64, vp]),
            "sbn_oracle_pack24": (i32, [vp, vp, i64, i64, vp, vp]),
            "sbn_oracle_unpack24": (None, [vp, vp, i64, i64, vp, vp]),
            "sbn_oracle_pack_vals2": (i32, [vp, i64, i64, vp]),
            "sbn_oracle_unpack_vals2": (i32, [vp, i64, i64, vp]),
            "sbn_oracle_quantize_mask_pack": (i32, [vp, i64, i64, vp, vp, vp, vp, vp, vp]),
            "sbn_oracle_quant_act": (None, [vp, i64, i64, vp, vp]),
            "sbn_oracle_norm_quant_act": (None, [vp, i64, i64, vp, f32, vp, vp, vp, vp]),
            "sbn_oracle_acc_dense": (None, [vp, vp, i64, i64, i64, vp]),
            "sbn_oracle_acc_packed": (None, [vp, vp, vp, i64, i64, i64, vp]),
            "sbn_oracle_acc_packed_sampled": (None, [vp, vp, vp, i64, i64, vp, vp, i64, vp]),
            "sbn_oracle_acc_dense_sampled": (None, [vp, vp, i64, i64, vp, vp, i64, vp]),
            "sbn_oracle_dequant": (None, [vp, f32, vp, vp, i64, i64, vp]),
            "sbn_oracle_f32_to_bf16": (None, [vp, i64, vp]),
            "sbn_oracle_flip_count": (ctypes.c_uint64, [vp, vp, i64, i64]),
            "sbn_oracle_num_threads": (i32, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError(f"expected {np.dtype(dtype)}, got {a.dtype}")
    return a


def num_threads() -> int:
    return int(_load().sbn_oracle_num_threads())


# -- Eq. 1: scale -------------------------------------------------------------------------------
def absmean_scale(W):
    """gamma = mean|W| (double accumulation), scale = max(gamma, 1e-5).  Returns
    (gamma, scale, near_tie) with near_tie True when another summation order rounds differently."""
    W = _c(W, np.float32)
    N, K = W.shape
    g = np.zeros(1, np.float32)
    s = np.zeros(1, np.float32)
    nt = np.zeros(1, np.int32)
    _load().sbn_oracle_absmean_scale(_p(W), N, K, _p(g), _p(s), _p(nt))
    return np.float32(g[0]), np.float32(s[0]), bool(nt[0])


# -- Eq. 2: mask --------------------------------------------------------------------------------
def nm_mask(W, n_keep=2, m_group=4):
    """Per-group top-n_keep-of-m_group indicator of |W| along the input dimension."""
    W = _c(W, np.float32)
    N, K = W.shape
    if K % m_group:
        raise ValueError("K must be a multiple of the group size")
    mask = np.zeros((N, K), np.uint8)
    _load().sbn_oracle_nm_mask(_p(W), N, K, int(n_keep), int(m_group), _p(mask))
    return mask


# -- Eq. 1: ternarise ---------------------------------------------------------------------------
def ternarize(W, scale):
    W = _c(W, np.float32)
    N, K = W.shape
    q = np.zeros((N, K), np.int8)
    _load().sbn_oracle_ternarize(_p(W), N, K, float(np.float32(scale)), _p(q))
    return q


# -- Eq. 3 --------------------------------------------------------------------------------------
def apply_mask(q, mask):
    q = _c(q, np.int8)
    mask = _c(mask, np.uint8)
    N, K = q.shape
    out = np.zeros((N, K), np.int8)
    _load().sbn_oracle_apply_mask(_p(q), _p(mask), N, K, _p(out))
    return out


def pack24(q, mask):
    q = _c(q, np.int8)
    mask = _c(mask, np.uint8)
    N, K = q.shape
    vals = np.zeros((N, K // 2), np.int8)
    meta = np.zeros((N, K // 8), np.uint8)
    rc = _load().sbn_oracle_pack24(_p(q), _p(mask), N, K, _p(vals), _p(meta))
    if rc != 0:
        raise ValueError("mask is not an exact 2:4 mask (or K % 8 != 0)")
    return vals, meta


def unpack24(vals, meta):
    vals = _c(vals, np.int8)
    meta = _c(meta, np.uint8)
    N, K2 = vals.shape
    K = 2 * K2
    weff = np.zeros((N, K), np.int8)
    mask = np.zeros((N, K), np.uint8)
    _load().sbn_oracle_unpack24(_p(vals), _p(meta), N, K, _p(weff), _p(mask))
    return weff, mask


def pack_vals2(vals):
    """Kept values int8 [N][K/2] -> two bits each (t = v + 1), uint8 [N][K/8]: the two values of a
    group in one nibble (t0 | t1 << 2), even groups in the low nibble of their byte."""
    vals = _c(vals, np.int8)
    N, K2 = vals.shape
    K = 2 * K2
    out = np.zeros((N, K // 8), np.uint8)
    if _load().sbn_oracle_pack_vals2(_p(vals), N, K, _p(out)) != 0:
        raise ValueError("values are not ternary (or K % 8 != 0)")
    return out


def unpack_vals2(vals2):
    vals2 = _c(vals2, np.uint8)
    N, K8 = vals2.shape
    K = 8 * K8
    vals = np.zeros((N, K // 2), np.int8)
    if _load().sbn_oracle_unpack_vals2(_p(vals2), N, K, _p(vals)) != 0:
        raise ValueError("illegal field value 3")
    return vals


def quantize_mask_pack(W):
    """Part 1 of the path.  Returns a dict: vals, meta, scale, dense_q, mask, near_tie."""
    W = _c(W, np.float32)
    N, K = W.shape
    if K % 8:
        raise ValueError("K must be a multiple of 8")
    vals = np.zeros((N, K // 2), np.int8)
    meta = np.zeros((N, K // 8), np.uint8)
    scale = np.zeros(1, np.float32)
    dense_q = np.zeros((N, K), np.int8)
    mask = np.zeros((N, K), np.uint8)
    nt = np.zeros(1, np.int32)
    rc = _load().sbn_oracle_quantize_mask_pack(_p(W), N, K, _p(vals), _p(meta), _p(scale),
                                               _p(dense_q), _p(mask), _p(nt))
    if rc != 0:
        raise RuntimeError("oracle pack failed")
    return dict(vals=vals, meta=meta, scale=np.float32(scale[0]), dense_q=dense_q, mask=mask,
                near_tie=bool(nt[0]))


def quantize_mask_nm(W, n_keep, m_group):
    """Eq. 1-3 for a general N:M pattern (Sec. 2.2; 6:8 is the pattern of the paper's main
    results): gamma and W_q from the DENSE matrix, the mask from the pre-quantised |W|,
    W_eff = W_q (.) M.  No packed form: the paper fixes none, so parity is on W_eff and the mask.
    Returns a dict: scale, mask, w_eff."""
    W = _c(W, np.float32)
    _, scale, _ = absmean_scale(W)
    mask = nm_mask(W, n_keep, m_group)
    w_eff = apply_mask(ternarize(W, scale), mask)
    return dict(scale=scale, mask=mask, w_eff=w_eff)


def nm_bitlinear(xq, a_scale, w_eff, scale, bias=None):
    """Eq. 4 with W_eff given element by element (any N:M pattern): (y fp32 [T][N], acc int32)."""
    acc = acc_dense(xq, w_eff)
    return dequant(acc, scale, a_scale, bias), acc


# -- activations ---------------------------------------------------------------------------------
def quant_act(x_bf16_bits):
    """x given as uint16 bf16 bit patterns [T][K]; returns (xq int8 [T][K], a_scale fp32 [T])."""
    x = _c(x_bf16_bits, np.uint16)
    T, K = x.shape
    xq = np.zeros((T, K), np.int8)
    a_scale = np.zeros(T, np.float32)
    _load().sbn_oracle_quant_act(_p(x), T, K, _p(xq), _p(a_scale))
    return xq, a_scale


def norm_quant_act(x_bf16_bits, g=None, eps=1e-6, want_xn=False):
    """Algorithm 1's x~ = Q_a(Norm(x)), Norm read as RMSNorm with gain g (None = ones).
    Returns dict(xq int8 [T][K], a_scale fp32 [T], near_tie bool [T][, xn fp32 [T][K]])."""
    x = _c(x_bf16_bits, np.uint16)
    T, K = x.shape
    gg = None if g is None else _c(g, np.float32)
    xq = np.zeros((T, K), np.int8)
    a_scale = np.zeros(T, np.float32)
    near = np.zeros(T, np.uint8)
    xn = np.zeros((T, K), np.float32) if want_xn else None
    _load().sbn_oracle_norm_quant_act(_p(x), T, K, _p(gg), ctypes.c_float(eps), _p(xq), _p(a_scale), _p(xn), _p(near))
    out = dict(xq=xq, a_scale=a_scale, near_tie=near.astype(bool))
    if want_xn:
        out["xn"] = xn
    return out


# -- Eq. 4 ---------------------------------------------------------------------------------------
def acc_dense(xq, Wmat):
    xq = _c(xq, np.int8)
    Wmat = _c(Wmat, np.int8)
    T, K = xq.shape
    N = Wmat.shape[0]
    acc = np.zeros((T, N), np.int32)
    _load().sbn_oracle_acc_dense(_p(xq), _p(Wmat), T, N, K, _p(acc))
    return acc


def acc_packed(xq, vals, meta):
    xq = _c(xq, np.int8)
    vals = _c(vals, np.int8)
    meta = _c(meta, np.uint8)
    T, K = xq.shape
    N = vals.shape[0]
    acc = np.zeros((T, N), np.int32)
    _load().sbn_oracle_acc_packed(_p(xq), _p(vals), _p(meta), T, N, K, _p(acc))
    return acc


def acc_packed_sampled(xq, vals, meta, t_idx, n_idx):
    xq = _c(xq, np.int8)
    vals = _c(vals, np.int8)
    meta = _c(meta, np.uint8)
    t_idx = _c(t_idx, np.int64)
    n_idx = _c(n_idx, np.int64)
    T, K = xq.shape
    N = vals.shape[0]
    acc = np.zeros(len(t_idx), np.int32)
    _load().sbn_oracle_acc_packed_sampled(_p(xq), _p(vals), _p(meta), N, K, _p(t_idx), _p(n_idx),
                                          len(t_idx), _p(acc))
    return acc


def acc_dense_sampled(xq, Wmat, t_idx, n_idx):
    xq = _c(xq, np.int8)
    Wmat = _c(Wmat, np.int8)
    t_idx = _c(t_idx, np.int64)
    n_idx = _c(n_idx, np.int64)
    T, K = xq.shape
    N = Wmat.shape[0]
    acc = np.zeros(len(t_idx), np.int32)
    _load().sbn_oracle_acc_dense_sampled(_p(xq), _p(Wmat), N, K, _p(t_idx), _p(n_idx),
                                         len(t_idx), _p(acc))
    return acc


def dequant(acc, scale, a_scale, bias=None):
    acc = _c(acc, np.int32)
    a_scale = _c(a_scale, np.float32)
    if bias is not None:
        bias = _c(bias, np.float32)
    T, N = acc.shape
    y = np.zeros((T, N), np.float32)
    _load().sbn_oracle_dequant(_p(acc), float(np.float32(scale)), _p(a_scale), _p(bias), T, N,
                               _p(y))
    return y


def f32_to_bf16_bits(y):
    y = _c(y, np.float32)
    out = np.zeros(y.shape, np.uint16)
    _load().sbn_oracle_f32_to_bf16(_p(y), y.size, _p(out))
    return out


def flip_count(mask_a, mask_b):
    mask_a = _c(mask_a, np.uint8)
    mask_b = _c(mask_b, np.uint8)
    N, K = mask_a.shape
    return int(_load().sbn_oracle_flip_count(_p(mask_a), _p(mask_b), N, K))


def sparse_bitlinear(xq, a_scale, vals, meta, scale, bias=None):
    """Eq. 4 from the compressed layout: returns (y fp32 [T][N], acc int32 [T][N])."""
    acc = acc_packed(xq, vals, meta)
    return dequant(acc, scale, a_scale, bias), acc


def bitlinear(xq, a_scale, dense_q, scale, bias=None):
    """Dense BitLinear (Sec. 2.1): returns (y, acc)."""
    acc = acc_dense(xq, dense_q)
    return dequant(acc, scale, a_scale, bias), acc


# ------------------------------------------------------------------------------------------------
# Backward of the layer under the dual straight-through estimator (Sec. 2.3, Eq. 5: the mask and the
# quantiser are both transparent to the gradient; Algorithm 1, "Backward"; Algorithm 2's backward,
# which returns g_out unchanged, so the weight gradient is the plain, DENSE gradient of F.linear).
#
# With y = F.linear(x_q, w_masked), x_q = x~ * a_scale[t] the fake-quantised activations and
# w_masked = W_eff * scale, autograd of the linear map gives
#     dW[n][k] = sum_t dY[t][n] * x_q[t][k]         -- reaches every master weight, pruned ones too
#     dX[t][k] = sum_n dY[t][n] * w_masked[n][k]    -- through Q_a as the identity
# Precision (the paper names none; its models are trained with bf16 tensors): dY arrives in bf16, the
# two saved operands are rounded to bf16 as a bf16 training run holds them, x_q_b = bf16(x~ * a_scale)
# and w_b = W_eff * bf16(scale) (exact, W_eff is ternary); the sums below are over those values, here
# in float64 (numpy matmul), so what the kernels may differ by is their fp32 accumulation order only.
# ------------------------------------------------------------------------------------------------
def bf16_bits_to_f64(bits):
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def bf16_round(a):
    """fp32 array -> the nearest bf16 values (ties to even), returned as float64."""
    return bf16_bits_to_f64(f32_to_bf16_bits(np.ascontiguousarray(a, dtype=np.float32)))


def fake_quant_act_bf16(xq, a_scale):
    """x_q_b[t][k] = bf16(float(x~[t][k]) * a_scale[t]) -- one fp32 product, one rounding."""
    xq = _c(xq, np.int8)
    a_scale = _c(a_scale, np.float32)
    return bf16_round(xq.astype(np.float32) * a_scale[:, None])


def backward_dw(dy_bf16_bits, xq, a_scale):
    """Eq. 5 / Algorithm 2's backward: dW = dY^T x_q_b, dense [N][K] (float64)."""
    dY = bf16_bits_to_f64(dy_bf16_bits)
    return dY.T @ fake_quant_act_bf16(xq, a_scale)


def backward_dx(dy_bf16_bits, w_eff, scale):
    """dX = dY w_b with w_b = W_eff * bf16(scale): [T][K] (float64)."""
    dY = bf16_bits_to_f64(dy_bf16_bits)
    s_b = float(bf16_round(np.array([scale], np.float32))[0])
    return (dY @ _c(w_eff, np.int8).astype(np.float64)) * s_b


def backward_dual_ste(dy_bf16_bits, xq, a_scale, w_eff, scale):
    """Both gradients of one Sparse-BitLinear layer: (dX [T][K], dW [N][K]) in float64."""
    return backward_dx(dy_bf16_bits, w_eff, scale), backward_dw(dy_bf16_bits, xq, a_scale)
