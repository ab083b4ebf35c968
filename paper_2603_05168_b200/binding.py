"""Thin ctypes binding over libsbn.so -- argument marshalling only.

Function names match the C ABI in ``include/sbn.h``.  Tensors are torch CUDA tensors used purely
as device buffers (``data_ptr()``), the stream is torch's current stream.  Nothing here computes:
every step of the path runs inside the library's kernels.  If the library cannot be loaded the
import of this module's functions fails loudly -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsbn.so")

SBN_OK = 0
OUT_F32, OUT_BF16 = 0, 1
OP_QUANTIZE_MASK_PACK, OP_QUANT_ACT, OP_SPARSE_BITLINEAR, OP_BITLINEAR, OP_BACKWARD = 0, 1, 2, 3, 4

EXPORTS = [
    "sbn_workspace_bytes", "sbn_xq_bytes", "sbn_quantize_mask_pack", "sbn_quantize_mask_pack_bf16", "sbn_quantize_mask_pack_static_ws", "sbn_quantize_mask_pack_batched",
    "sbn_batch_workspace_bytes", "sbn_quant_act", "sbn_quant_act_expand68", "sbn_expanded_k", "sbn_norm_quant_act", "sbn_norm_quant_act_expand68", "sbn_sparse_bitlinear", "sbn_pack_vals2", "sbn_sparse_bitlinear_packed", "sbn_quant_act_sparse_bitlinear", "sbn_quant_act_bitlinear",
    "sbn_bitlinear", "sbn_layer_forward_host", "sbn_check_status", "sbn_status_string",
    "sbn_set_gemm_tuning", "sbn_plan_gemm", "sbn_launch_count", "sbn_unpack_canonical", "sbn_tile_canonical",
    "sbn_set_wait_test", "sbn_set_gemm_probe", "sbn_bitlinear_backward",
]

_lib = None


class SbnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: sbn status {code} ({status_string(code)})")


def lib() -> ctypes.CDLL:
    """Load libsbn.so (built in-tree by paper_2603_05168_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2603_05168_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.sbn_xq_bytes.restype = sz
        L.sbn_xq_bytes.argtypes = [i32, i32]
        L.sbn_workspace_bytes.restype = sz
        L.sbn_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.sbn_quantize_mask_pack.restype = i32
        L.sbn_quantize_mask_pack.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.sbn_quantize_mask_pack_bf16.restype = i32
        L.sbn_quantize_mask_pack_bf16.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.sbn_quantize_mask_pack_static_ws.restype = i32
        L.sbn_quantize_mask_pack_static_ws.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.sbn_batch_workspace_bytes.restype = sz
        L.sbn_batch_workspace_bytes.argtypes = [i32]
        L.sbn_quantize_mask_pack_batched.restype = i32
        L.sbn_quantize_mask_pack_batched.argtypes = [i32, vp, vp, sz, vp]
        L.sbn_quant_act.restype = i32
        L.sbn_quant_act.argtypes = [vp, i32, i32, vp, vp, vp]
        L.sbn_quant_act_expand68.restype = i32
        L.sbn_quant_act_expand68.argtypes = [vp, i32, i32, vp, vp, vp]
        L.sbn_expanded_k.restype = i32
        L.sbn_expanded_k.argtypes = [i32, i32, i32]
        L.sbn_norm_quant_act.restype = i32
        L.sbn_norm_quant_act.argtypes = [vp, i32, i32, vp, ctypes.c_float, vp, vp, vp]
        L.sbn_norm_quant_act_expand68.restype = i32
        L.sbn_norm_quant_act_expand68.argtypes = [vp, i32, i32, vp, ctypes.c_float, vp, vp, vp]
        L.sbn_sparse_bitlinear.restype = i32
        L.sbn_sparse_bitlinear.argtypes = [vp, vp, i32, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp, sz, vp]
        L.sbn_quant_act_sparse_bitlinear.restype = i32
        L.sbn_quant_act_sparse_bitlinear.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp, vp]
        L.sbn_quant_act_bitlinear.restype = i32
        L.sbn_quant_act_bitlinear.argtypes = [vp, i32, vp, vp, i32, i32, vp, vp, i32, vp, vp, vp]
        L.sbn_pack_vals2.restype = i32
        L.sbn_pack_vals2.argtypes = [vp, i32, i32, vp, vp]
        L.sbn_sparse_bitlinear_packed.restype = i32
        L.sbn_sparse_bitlinear_packed.argtypes = [vp, vp, i32, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp]
        L.sbn_bitlinear.restype = i32
        L.sbn_bitlinear.argtypes = [vp, vp, i32, vp, vp, i32, i32, vp, vp, i32, vp, vp, sz, vp]
        L.sbn_layer_forward_host.restype = i32
        L.sbn_layer_forward_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, i32, vp, sz, vp]
        L.sbn_check_status.restype = i32
        L.sbn_check_status.argtypes = [vp]
        L.sbn_status_string.restype = ctypes.c_char_p
        L.sbn_status_string.argtypes = [i32]
        L.sbn_set_gemm_tuning.restype = None
        L.sbn_set_gemm_tuning.argtypes = [i32, i32]
        L.sbn_plan_gemm.restype = None
        L.sbn_plan_gemm.argtypes = [i32, i32, i32, i32, vp]
        L.sbn_unpack_canonical.restype = i32
        L.sbn_unpack_canonical.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.sbn_tile_canonical.restype = i32
        L.sbn_tile_canonical.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.sbn_bitlinear_backward.restype = i32
        L.sbn_bitlinear_backward.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, sz, vp]
        L.sbn_set_gemm_probe.restype = None
        L.sbn_set_gemm_probe.argtypes = [i32]
        L.sbn_set_wait_test.restype = i32
        L.sbn_set_wait_test.argtypes = [i32, ctypes.c_ulonglong]
        L.sbn_launch_count.restype = ctypes.c_ulonglong
        L.sbn_launch_count.argtypes = []
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sbn_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != SBN_OK:
        raise SbnError(code, where)


def sbn_workspace_bytes(op: int, T: int, N: int, K: int) -> int:
    return int(lib().sbn_workspace_bytes(op, T, N, K))


def sbn_xq_bytes(T: int, K: int) -> int:
    return int(lib().sbn_xq_bytes(T, K))


def sbn_quantize_mask_pack(W, vals, meta, w_scale, ws, dense_q=None, prev_meta=None, flip_bits=None,
                           n_keep: int = 2, m_group: int = 4):
    """W: fp32 or bf16 CUDA tensor [N][K] (bf16 master weights go to sbn_quantize_mask_pack_bf16)."""
    N, K = W.shape
    fn = lib().sbn_quantize_mask_pack_bf16 if W.dtype == torch.bfloat16 else lib().sbn_quantize_mask_pack
    _check(fn(_ptr(W), N, K, n_keep, m_group, _ptr(vals), _ptr(meta),
              _ptr(w_scale), _ptr(dense_q), _ptr(prev_meta), _ptr(flip_bits),
              _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "sbn_quantize_mask_pack")


def sbn_quantize_mask_pack_static_ws(W, vals, meta, w_scale, dense_q=None, prev_meta=None, flip_bits=None,
                                     n_keep: int = 2, m_group: int = 4):
    """Workspace-free variant: the scratch is a fixed array inside the library (see sbn.h for
    its limits and the rule about overlapping calls)."""
    N, K = W.shape
    _check(lib().sbn_quantize_mask_pack_static_ws(_ptr(W), N, K, n_keep, m_group, _ptr(vals), _ptr(meta),
                                                  _ptr(w_scale), _ptr(dense_q), _ptr(prev_meta),
                                                  _ptr(flip_bits), _stream()),
           "sbn_quantize_mask_pack_static_ws")


class PackJob(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("N", ctypes.c_int), ("K", ctypes.c_int), ("vals", ctypes.c_void_p),
                ("meta", ctypes.c_void_p), ("w_scale", ctypes.c_void_p), ("dense_q", ctypes.c_void_p),
                ("prev_meta", ctypes.c_void_p), ("flip_bits", ctypes.c_void_p), ("w_bf16", ctypes.c_int),
                ("gamma_hint", ctypes.c_void_p)]


def sbn_batch_workspace_bytes(count: int) -> int:
    return int(lib().sbn_batch_workspace_bytes(int(count)))


def make_pack_jobs(jobs):
    """jobs: list of dicts with W, vals, meta, w_scale and optionally dense_q, prev_meta, flip_bits,
    gamma_hint (torch CUDA tensors).  Returns the ctypes array to hand to sbn_quantize_mask_pack_batched; it can
    be reused every step as long as the tensors stay where they are."""
    arr = (PackJob * len(jobs))()
    for a, j in zip(arr, jobs):
        N, K = j["W"].shape
        a.W, a.N, a.K = j["W"].data_ptr(), N, K
        a.w_bf16 = 1 if j["W"].dtype == torch.bfloat16 else 0
        a.vals, a.meta, a.w_scale = j["vals"].data_ptr(), j["meta"].data_ptr(), j["w_scale"].data_ptr()
        for key in ("dense_q", "prev_meta", "flip_bits", "gamma_hint"):
            t = j.get(key)
            setattr(a, key, t.data_ptr() if t is not None else None)
    return arr


def sbn_quantize_mask_pack_batched(job_array, ws):
    _check(lib().sbn_quantize_mask_pack_batched(len(job_array), ctypes.cast(job_array, ctypes.c_void_p), _ptr(ws),
                                                ws.numel() * ws.element_size(), _stream()),
           "sbn_quantize_mask_pack_batched")


def sbn_quant_act(x_bf16, xq, a_scale):
    T, K = x_bf16.shape
    _check(lib().sbn_quant_act(_ptr(x_bf16), T, K, _ptr(xq), _ptr(a_scale), _stream()), "sbn_quant_act")


def sbn_quant_act_expand68(x_bf16, xq, a_scale):
    T, K = x_bf16.shape
    _check(lib().sbn_quant_act_expand68(_ptr(x_bf16), T, K, _ptr(xq), _ptr(a_scale), _stream()),
           "sbn_quant_act_expand68")


def sbn_expanded_k(K: int, n_keep: int, m_group: int) -> int:
    return int(lib().sbn_expanded_k(K, n_keep, m_group))


def sbn_norm_quant_act(x_bf16, xq, a_scale, gain=None, eps: float = 1e-6, expand68: bool = False):
    T, K = x_bf16.shape
    fn = lib().sbn_norm_quant_act_expand68 if expand68 else lib().sbn_norm_quant_act
    _check(fn(_ptr(x_bf16), T, K, _ptr(gain), ctypes.c_float(eps), _ptr(xq), _ptr(a_scale), _stream()),
           "sbn_norm_quant_act")


def _ws_args(ws):
    if ws is None:
        return None, 0
    return _ptr(ws), ws.numel() * ws.element_size()


def sbn_sparse_bitlinear(xq, a_scale, vals, meta, w_scale, y, bias=None, acc_out=None, ws=None):
    T, N = y.shape
    K = 2 * vals.numel() // N
    dt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    wp, wb = _ws_args(ws)
    _check(lib().sbn_sparse_bitlinear(_ptr(xq), _ptr(a_scale), T, _ptr(vals), _ptr(meta), _ptr(w_scale),
                                      N, K, _ptr(bias), _ptr(y), dt, _ptr(acc_out), wp, wb, _stream()),
           "sbn_sparse_bitlinear")


def sbn_quant_act_sparse_bitlinear(x_bf16, vals, meta, w_scale, y, bias=None, acc_out=None, a_scale_out=None):
    """Activation quantiser + sparse GEMM in one kernel (few tokens)."""
    T, K = x_bf16.shape
    N = y.shape[1]
    dt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    _check(lib().sbn_quant_act_sparse_bitlinear(_ptr(x_bf16), T, _ptr(vals), _ptr(meta), _ptr(w_scale), N, K, _ptr(bias),
                                                _ptr(y), dt, _ptr(acc_out), _ptr(a_scale_out), _stream()),
           "sbn_quant_act_sparse_bitlinear")


def sbn_quant_act_bitlinear(x_bf16, dense_q, w_scale, y, bias=None, acc_out=None, a_scale_out=None):
    T, K = x_bf16.shape
    N = y.shape[1]
    dt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    _check(lib().sbn_quant_act_bitlinear(_ptr(x_bf16), T, _ptr(dense_q), _ptr(w_scale), N, K, _ptr(bias), _ptr(y), dt,
                                         _ptr(acc_out), _ptr(a_scale_out), _stream()),
           "sbn_quant_act_bitlinear")


def sbn_pack_vals2(vals, vals2):
    N = vals.shape[0]
    K = 2 * vals.numel() // N
    _check(lib().sbn_pack_vals2(_ptr(vals), N, K, _ptr(vals2), _stream()), "sbn_pack_vals2")


def sbn_sparse_bitlinear_packed(xq, a_scale, vals2, meta, w_scale, y, bias=None, acc_out=None):
    T, N = y.shape
    K = 8 * vals2.numel() // N
    dt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    _check(lib().sbn_sparse_bitlinear_packed(_ptr(xq), _ptr(a_scale), T, _ptr(vals2), _ptr(meta), _ptr(w_scale), N, K,
                                             _ptr(bias), _ptr(y), dt, _ptr(acc_out), _stream()),
           "sbn_sparse_bitlinear_packed")


def alloc_vals2(N: int, K: int, device="cuda"):
    """Device buffer for the kept values at two bits each ([N][K/8] bytes, tiled like meta)."""
    return torch.empty((N, K // 8), dtype=torch.uint8, device=device)


def sbn_bitlinear(xq, a_scale, dense_q, w_scale, y, bias=None, acc_out=None, ws=None):
    T, N = y.shape
    K = dense_q.numel() // N
    dt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    wp, wb = _ws_args(ws)
    _check(lib().sbn_bitlinear(_ptr(xq), _ptr(a_scale), T, _ptr(dense_q), _ptr(w_scale), N, K,
                               _ptr(bias), _ptr(y), dt, _ptr(acc_out), wp, wb, _stream()),
           "sbn_bitlinear")


def sbn_layer_forward_host(x_host, x_dev, xq_dev, a_scale_dev, w_scale, y_dev, y_host, vals=None,
                           meta=None, dense_q=None, bias=None, ws=None):
    """x_host / y_host are (pinned) CPU tensors; everything else lives on the device."""
    T, K = x_host.shape
    N = y_host.shape[1]
    dt = OUT_BF16 if y_host.dtype == torch.bfloat16 else OUT_F32
    wp, wb = _ws_args(ws)
    _check(lib().sbn_layer_forward_host(_ptr(x_host), T, K, _ptr(x_dev), _ptr(xq_dev), _ptr(a_scale_dev),
                                        _ptr(vals), _ptr(meta), _ptr(dense_q), _ptr(w_scale), N,
                                        _ptr(bias), _ptr(y_dev), _ptr(y_host), dt, wp, wb, _stream()),
           "sbn_layer_forward_host")


def sbn_unpack_canonical(vals, meta, N: int, K: int, vals_out, meta_out):
    """Tiled vals / meta -> plain row-major [N][K/2] / [N][K/8] (either pair may be None)."""
    _check(lib().sbn_unpack_canonical(_ptr(vals), _ptr(meta), N, K, _ptr(vals_out), _ptr(meta_out), _stream()),
           "sbn_unpack_canonical")


def sbn_tile_canonical(vals_plain, meta_plain, N: int, K: int, vals, meta):
    """Plain row-major vals / meta -> the library's tiled order (either pair may be None)."""
    _check(lib().sbn_tile_canonical(_ptr(vals_plain), _ptr(meta_plain), N, K, _ptr(vals), _ptr(meta), _stream()),
           "sbn_tile_canonical")


def sbn_set_wait_test(break_waits: bool = False, wait_limit_us: int = 0):
    _check(lib().sbn_set_wait_test(1 if break_waits else 0, int(wait_limit_us)), "sbn_set_wait_test")


def sbn_bitlinear_backward(dY, xq, a_scale, vals, meta, w_scale, N: int, K: int, dX=None, dW=None, ws=None):
    """Dual-STE backward of one layer: dX (bf16 [T][K]) and / or dW (fp32 [N][K]) from dY (bf16 [T][N])."""
    T = dY.shape[0]
    wp, wb = _ws_args(ws)
    _check(lib().sbn_bitlinear_backward(_ptr(dY), T, _ptr(xq), _ptr(a_scale), _ptr(vals), _ptr(meta), _ptr(w_scale), N, K,
                                        _ptr(dX), _ptr(dW), wp, wb, _stream()),
           "sbn_bitlinear_backward")


def sbn_set_gemm_probe(flags: int = 0):
    """Timing experiments on the CTA-pair GEMM (results are wrong while flags != 0); see sbn.h."""
    lib().sbn_set_gemm_probe(int(flags))


def sbn_check_status():
    _check(lib().sbn_check_status(_stream()), "sbn_check_status")


def sbn_set_gemm_tuning(token_tile: int = 0, split_k: int = 0):
    lib().sbn_set_gemm_tuning(int(token_tile), int(split_k))


def sbn_plan_gemm(sparse: bool, T: int, N: int, K: int):
    """(kernel, tokens per tile, split-K factor, cluster size) the dispatcher picks; launches nothing."""
    out = (ctypes.c_int * 4)()
    lib().sbn_plan_gemm(1 if sparse else 0, T, N, K, out)
    return tuple(out)


def sbn_launch_count() -> int:
    return int(lib().sbn_launch_count())


# -- small conveniences for callers (allocation only) ---------------------------------------------
def alloc_packed(N: int, K: int, device="cuda", with_dense: bool = False, n_keep: int = 2, m_group: int = 4):
    """Device buffers for one packed weight matrix (for 6:8: the 2:4 form over K' = 3K/2 columns)."""
    Kp = sbn_expanded_k(K, n_keep, m_group)
    if Kp == 0:
        raise ValueError(f"unsupported pattern {n_keep}:{m_group} for K = {K}")
    out = dict(
        vals=torch.empty((N, Kp // 2), dtype=torch.int8, device=device),
        meta=torch.empty((N, Kp // 8), dtype=torch.uint8, device=device),
        w_scale=torch.empty(1, dtype=torch.float32, device=device),
        ws=torch.empty(sbn_workspace_bytes(OP_QUANTIZE_MASK_PACK, 0, N, K), dtype=torch.uint8, device=device),
    )
    if with_dense:
        out["dense_q"] = torch.empty((N, K), dtype=torch.int8, device=device)
    return out


def alloc_xq(T: int, K: int, device="cuda"):
    """Device buffer for the tiled int8 activations of T tokens x K columns."""
    return torch.empty(sbn_xq_bytes(T, K), dtype=torch.int8, device=device)


def alloc_gemm_ws(op: int, T: int, N: int, K: int, device="cuda"):
    n = sbn_workspace_bytes(op, T, N, K)
    return torch.zeros(max(n, 16), dtype=torch.uint8, device=device)      # zero-filled once, kept zero by the library
