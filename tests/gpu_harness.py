"""Helpers for the GPU parity tests: move seeded numpy inputs to the device, call the library
through its binding, bring results back as numpy arrays."""
import numpy as np
import torch

from paper_2603_05168_b200 import binding as b


# ---- the library's tiled storage orders, restated from the formulas documented in include/sbn.h --
def _vals_offsets(N, K):
    n = np.arange(N, dtype=np.int64)[:, None]
    c = np.arange(K // 2, dtype=np.int64)[None, :]
    KB, r, cc = K // 128, n & 127, c & 63
    return ((n >> 7) * KB + (c >> 6)) * 8192 + (r << 6) + ((((cc >> 4) ^ ((r >> 1) & 3))) << 4) + (cc & 15)


def _meta_offsets(N, K):
    n = np.arange(N, dtype=np.int64)[:, None]
    b = np.arange(K // 8, dtype=np.int64)[None, :]
    KB, r = K // 128, n & 127
    return ((n >> 7) * KB + (b >> 4)) * 2048 + (r << 4) + (b & 15)


def _dense_offsets(N, K):
    n = np.arange(N, dtype=np.int64)[:, None]
    k = np.arange(K, dtype=np.int64)[None, :]
    KB, r, c = K // 128, n & 127, k & 127
    return ((n >> 7) * KB + (k >> 7)) * 16384 + ((r >> 3) << 10) + ((r & 7) << 7) + ((((c >> 4) ^ (r & 7))) << 4) + (c & 15)


def _xq_offsets(T, K):
    t = np.arange(T, dtype=np.int64)[:, None]
    k = np.arange(K, dtype=np.int64)[None, :]
    TB8, r, c = 2 * ((T + 15) // 16), t & 7, k & 127
    return ((k >> 7) * TB8 + (t >> 3)) * 1024 + (r << 7) + ((((c >> 4) ^ r)) << 4) + (c & 15)


def untile(flat: np.ndarray, offsets: np.ndarray) -> np.ndarray:
    """tiled byte buffer -> plain row-major array."""
    return np.ascontiguousarray(flat.reshape(-1)[offsets])


def tile(canonical: np.ndarray, offsets: np.ndarray, nbytes: int) -> np.ndarray:
    """plain row-major array -> tiled byte buffer (bytes no element maps to stay 0)."""
    out = np.zeros(nbytes, canonical.dtype)
    out[offsets] = canonical
    return out


def tile_vals(vals):
    N, K2 = vals.shape
    return tile(vals, _vals_offsets(N, 2 * K2), vals.size)


def tile_meta(meta):
    N, K8 = meta.shape
    return tile(meta, _meta_offsets(N, 8 * K8), meta.size)


def tile_xq(xq):
    T, K = xq.shape
    return tile(xq, _xq_offsets(T, K), b.sbn_xq_bytes(T, K))


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def gpu_quantize_mask_pack(W: np.ndarray, with_dense=True, prev_meta=None, in_place=False, w_bf16_bits=None):
    """W fp32 [N][K]; or, with w_bf16_bits (uint16 bit patterns), bf16 master weights."""
    N, K = W.shape
    bufs = b.alloc_packed(N, K, with_dense=with_dense)
    Wd = dev(W) if w_bf16_bits is None else bf16_dev(w_bf16_bits)
    flip = None
    pm = None
    if prev_meta is not None:
        flip = torch.full((1,), 12345, dtype=torch.int64, device="cuda")   # must be overwritten
        prev_tiled = tile_meta(prev_meta).reshape(N, K // 8)
        if in_place:
            bufs["meta"].copy_(dev(prev_tiled))
            pm = bufs["meta"]
        else:
            pm = dev(prev_tiled)
    b.sbn_quantize_mask_pack(Wd, bufs["vals"], bufs["meta"], bufs["w_scale"], bufs["ws"],
                             dense_q=bufs.get("dense_q"), prev_meta=pm, flip_bits=flip)
    b.sbn_check_status()
    out = dict(vals=untile(bufs["vals"].cpu().numpy(), _vals_offsets(N, K)),
               meta=untile(bufs["meta"].cpu().numpy(), _meta_offsets(N, K)),
               scale=np.float32(bufs["w_scale"].cpu().numpy()[0]), dev=bufs)
    if with_dense:
        out["dense_q"] = untile(bufs["dense_q"].cpu().numpy(), _dense_offsets(N, K))
    if flip is not None:
        out["flips"] = int(flip.cpu().numpy()[0])
    return out


# ---- the 6:8 pattern: index maps between the K columns and the K' = 3K/2 expanded columns --------
def expand68_columns(K):
    """For every expanded column 12 g + 4 w + s the original column 8 g + 2 w + s (as documented in
    include/sbn.h)."""
    kp = np.arange(3 * K // 2, dtype=np.int64)
    g, rem = kp // 12, kp % 12
    return 8 * g + 2 * (rem // 4) + (rem % 4)


def fold68(mat_p):
    """[N][K'] array over the expanded columns -> [N][K]: sum of the (up to two) expanded columns that
    carry each original column."""
    N, Kp = mat_p.shape
    K = Kp * 2 // 3
    out = np.zeros((N, K), np.int64)
    np.add.at(out, (np.arange(N)[:, None], expand68_columns(K)[None, :]), mat_p.astype(np.int64))
    return out


def gpu_quantize_mask_pack68(W: np.ndarray, prev_meta=None, in_place=False, w_bf16_bits=None):
    """6:8 pack.  Returns the 2:4 form of the [N][K'] matrix in plain order (vals [N][K'/2],
    meta [N][K'/8]), the scale, the device buffers and, with prev_meta (plain [N][K'/8]), flips."""
    N, K = W.shape
    Kp = 3 * K // 2
    bufs = b.alloc_packed(N, K, n_keep=6, m_group=8)
    Wd = dev(W) if w_bf16_bits is None else bf16_dev(w_bf16_bits)
    flip = pm = None
    if prev_meta is not None:
        flip = torch.full((1,), 12345, dtype=torch.int64, device="cuda")
        prev_tiled = tile_meta(prev_meta).reshape(N, Kp // 8)
        if in_place:
            bufs["meta"].copy_(dev(prev_tiled))
            pm = bufs["meta"]
        else:
            pm = dev(prev_tiled)
    bufs["vals"].fill_(77)                                   # every byte must be written
    if not in_place:
        bufs["meta"].fill_(0xEE)
    b.sbn_quantize_mask_pack(Wd, bufs["vals"], bufs["meta"], bufs["w_scale"], bufs["ws"],
                             prev_meta=pm, flip_bits=flip, n_keep=6, m_group=8)
    b.sbn_check_status()
    out = dict(vals=untile(bufs["vals"].cpu().numpy(), _vals_offsets(N, Kp)),
               meta=untile(bufs["meta"].cpu().numpy(), _meta_offsets(N, Kp)),
               scale=np.float32(bufs["w_scale"].cpu().numpy()[0]), dev=bufs)
    if flip is not None:
        out["flips"] = int(flip.cpu().numpy()[0])
    return out


def gpu_quant_act_expand68(x_bits: np.ndarray):
    T, K = x_bits.shape
    xd = bf16_dev(x_bits)
    xq = b.alloc_xq(T, 3 * K // 2)
    xq.fill_(99)
    a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
    b.sbn_quant_act_expand68(xd, xq, a_scale)
    b.sbn_check_status()
    return xq, a_scale


def gpu_quant_act(x_bits: np.ndarray):
    T, K = x_bits.shape
    xd = bf16_dev(x_bits)
    xq = b.alloc_xq(T, K)
    a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
    b.sbn_quant_act(xd, xq, a_scale)
    b.sbn_check_status()
    return xq, a_scale


def gpu_norm_quant_act(x_bits: np.ndarray, gain=None, eps=1e-6, expand68=False):
    T, K = x_bits.shape
    xd = bf16_dev(x_bits)
    xq = b.alloc_xq(T, 3 * K // 2 if expand68 else K)
    xq.fill_(55)
    a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
    gd = None if gain is None else dev(np.asarray(gain, np.float32))
    b.sbn_norm_quant_act(xd, xq, a_scale, gain=gd, eps=eps, expand68=expand68)
    b.sbn_check_status()
    return xq, a_scale


def xq_to_numpy(xq: torch.Tensor, T: int, K: int) -> np.ndarray:
    """Tiled device activations -> plain [T][K] int8."""
    return untile(xq.cpu().numpy(), _xq_offsets(T, K))


def gpu_gemm(sparse: bool, xq, a_scale, packed_dev, out_dtype=torch.float32, bias=None, want_acc=True):
    """xq / a_scale: device tensors; packed_dev: dict of device tensors from alloc_packed."""
    T = a_scale.numel()
    N, K = packed_dev["vals"].shape[0], 2 * packed_dev["vals"].shape[1]
    y = torch.full((T, N), float("nan"), dtype=out_dtype, device="cuda")
    acc = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device="cuda") if want_acc else None
    op = b.OP_SPARSE_BITLINEAR if sparse else b.OP_BITLINEAR
    ws = b.alloc_gemm_ws(op, T, N, K)
    if sparse:
        b.sbn_sparse_bitlinear(xq, a_scale, packed_dev["vals"], packed_dev["meta"], packed_dev["w_scale"],
                               y, bias=bias, acc_out=acc, ws=ws)
    else:
        b.sbn_bitlinear(xq, a_scale, packed_dev["dense_q"], packed_dev["w_scale"], y, bias=bias,
                        acc_out=acc, ws=ws)
    b.sbn_check_status()
    return y, acc


def gpu_unpack_canonical(packed_dev, N, K):
    """The library's own un-tiling call: device vals / meta (tiled) -> plain [N][K/2] int8 and [N][K/8]
    uint8 numpy arrays.  No numpy permutation involved."""
    vals_out = torch.full((N, K // 2), 99, dtype=torch.int8, device="cuda")
    meta_out = torch.full((N, K // 8), 0xEE, dtype=torch.uint8, device="cuda")
    b.sbn_unpack_canonical(packed_dev["vals"], packed_dev["meta"], N, K, vals_out, meta_out)
    b.sbn_check_status()
    return vals_out.cpu().numpy(), meta_out.cpu().numpy()


def gpu_pack_vals2(packed_dev):
    """Device buffers of alloc_packed -> (device vals2 buffer, plain uint8 [N][K/8])."""
    N, K = packed_dev["vals"].shape[0], 2 * packed_dev["vals"].shape[1]
    out = b.alloc_vals2(N, K)
    out.fill_(0xAA)
    b.sbn_pack_vals2(packed_dev["vals"], out)
    b.sbn_check_status()
    return out, untile(out.cpu().numpy(), _meta_offsets(N, K))


def gpu_gemm_packed(xq, a_scale, vals2, packed_dev, out_dtype=torch.float32, bias=None, want_acc=True):
    T = a_scale.numel()
    N = packed_dev["vals"].shape[0]
    y = torch.full((T, N), float("nan"), dtype=out_dtype, device="cuda")
    acc = torch.full((T, N), -(2 ** 31), dtype=torch.int32, device="cuda") if want_acc else None
    b.sbn_sparse_bitlinear_packed(xq, a_scale, vals2, packed_dev["meta"], packed_dev["w_scale"], y, bias=bias, acc_out=acc)
    b.sbn_check_status()
    return y, acc


def y_to_f32_numpy(y: torch.Tensor) -> np.ndarray:
    return y.float().cpu().numpy()


def bf16_tensor_bits(y: torch.Tensor) -> np.ndarray:
    return y.view(torch.int16).cpu().numpy().view(np.uint16)
