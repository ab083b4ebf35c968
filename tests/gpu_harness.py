"""Helpers for the GPU parity tests: move seeded numpy inputs to the device, call the library
through its binding, bring results back as numpy arrays."""
import numpy as np
import torch

from paper_2603_05168_b200 import binding as b


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def gpu_quantize_mask_pack(W: np.ndarray, with_dense=True, prev_meta=None, in_place=False):
    N, K = W.shape
    bufs = b.alloc_packed(N, K, with_dense=with_dense)
    Wd = dev(W)
    flip = None
    pm = None
    if prev_meta is not None:
        flip = torch.full((1,), 12345, dtype=torch.int64, device="cuda")   # must be overwritten
        if in_place:
            bufs["meta"].copy_(dev(prev_meta))
            pm = bufs["meta"]
        else:
            pm = dev(prev_meta)
    b.sbn_quantize_mask_pack(Wd, bufs["vals"], bufs["meta"], bufs["w_scale"], bufs["ws"],
                             dense_q=bufs.get("dense_q"), prev_meta=pm, flip_bits=flip)
    b.sbn_check_status()
    out = dict(vals=bufs["vals"].cpu().numpy(), meta=bufs["meta"].cpu().numpy(),
               scale=np.float32(bufs["w_scale"].cpu().numpy()[0]), dev=bufs)
    if with_dense:
        out["dense_q"] = bufs["dense_q"].cpu().numpy()
    if flip is not None:
        out["flips"] = int(flip.cpu().numpy()[0])
    return out


def gpu_quant_act(x_bits: np.ndarray):
    T, K = x_bits.shape
    xd = bf16_dev(x_bits)
    xq = torch.empty((T, K), dtype=torch.int8, device="cuda")
    a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
    b.sbn_quant_act(xd, xq, a_scale)
    b.sbn_check_status()
    return xq, a_scale


def gpu_gemm(sparse: bool, xq, a_scale, packed_dev, out_dtype=torch.float32, bias=None, want_acc=True):
    """xq / a_scale: device tensors; packed_dev: dict of device tensors from alloc_packed."""
    T, K = xq.shape
    N = packed_dev["vals"].shape[0]
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


def y_to_f32_numpy(y: torch.Tensor) -> np.ndarray:
    return y.float().cpu().numpy()


def bf16_tensor_bits(y: torch.Tensor) -> np.ndarray:
    return y.view(torch.int16).cpu().numpy().view(np.uint16)
