"""CPU-only checks of the boundary: the library builds, loads, exports every symbol that
include/sbn.h declares, and rejects bad arguments on the host before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2603_05168_b200 import build as sbn_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    sbn_build.build()
    from paper_2603_05168_b200 import binding
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sbn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sbn_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    names = _declared_functions()
    assert {"sbn_quantize_mask_pack", "sbn_quant_act", "sbn_sparse_bitlinear", "sbn_bitlinear"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"{n} declared in sbn.h but not exported"
    from paper_2603_05168_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_status_strings(L):
    from paper_2603_05168_b200 import binding
    seen = {binding.status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert binding.status_string(99) == "unknown status"


def test_workspace_query(L):
    from paper_2603_05168_b200 import binding as b
    assert b.sbn_workspace_bytes(b.OP_QUANTIZE_MASK_PACK, 0, 256, 256) >= 8 * 148
    assert b.sbn_workspace_bytes(b.OP_QUANT_ACT, 64, 0, 256) == 0
    # large T: no split-K; few tokens: split-K inside clusters, reduced on chip -- no scratch either
    assert b.sbn_workspace_bytes(b.OP_SPARSE_BITLINEAR, 4096, 2560, 2560) == 0
    assert b.sbn_workspace_bytes(b.OP_SPARSE_BITLINEAR, 4, 2560, 2560) == 0
    # split-K through global memory (here forced): int32 [T][N] sums + one counter per output tile
    b.sbn_set_gemm_tuning(64, 5)
    try:
        assert b.sbn_workspace_bytes(b.OP_SPARSE_BITLINEAR, 4, 2560, 2560) == 4 * 2560 * 4 + 20 * 4
    finally:
        b.sbn_set_gemm_tuning(0, 0)
    assert b.sbn_workspace_bytes(b.OP_BITLINEAR, 4, 2560, 100) == 0      # illegal shape -> 0
    assert b.sbn_workspace_bytes(77, 4, 2560, 2560) == 0


def test_argument_validation_on_host(L):
    # fake, never dereferenced, 16-byte aligned "device pointers": every call below must return
    # an error code from the host-side checks before any CUDA call is made
    p = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1004)
    NULL, SHAPE, ALIGN, UNSUP, WS = 1, 2, 3, 4, 5
    assert L.sbn_quant_act(None, 4, 256, p, p, None) == NULL
    assert L.sbn_quant_act(p, 0, 256, p, p, None) == SHAPE
    assert L.sbn_quant_act(p, 4, 100, p, p, None) == SHAPE
    assert L.sbn_quant_act(odd, 4, 256, p, p, None) == ALIGN
    nq = lambda **k: L.sbn_norm_quant_act(k.get("x", p), k.get("T", 4), k.get("K", 256), k.get("g", p),
                                          ctypes.c_float(k.get("eps", 1e-6)), p, p, None)
    assert nq(x=None) == NULL
    assert nq(T=0) == SHAPE
    assert nq(K=100) == SHAPE
    assert nq(K=16384 + 128) == UNSUP           # row no longer fits in registers
    assert nq(eps=-1.0) == SHAPE
    assert nq(g=odd) == ALIGN
    assert nq(x=odd) == ALIGN
    qmp16 = lambda **k: L.sbn_quantize_mask_pack_bf16(k.get("W", p), k.get("N", 256), k.get("K", 256), k.get("n", 2),
                                                      k.get("m", 4), p, p, p, None, None, None, p, k.get("wsb", 1 << 20), None)
    assert qmp16(W=None) == NULL
    assert qmp16(n=5, m=8) == UNSUP
    assert qmp16(n=6, m=8, K=384) == SHAPE      # 6:8 needs K % 256 == 0
    assert qmp16(K=64) == SHAPE
    assert qmp16(wsb=8) == WS
    assert qmp16(W=odd) == ALIGN
    qmp = lambda **k: L.sbn_quantize_mask_pack(k.get("W", p), k.get("N", 256), k.get("K", 256), k.get("n", 2),
                                               k.get("m", 4), p, p, p, None, k.get("prev"), k.get("flip"),
                                               k.get("ws", p), k.get("wsb", 1 << 20), None)
    assert qmp(W=None) == NULL
    assert qmp(n=4, m=8) == UNSUP
    assert qmp(n=6, m=8, K=128) == SHAPE        # 6:8 needs K % 256 == 0
    assert L.sbn_quantize_mask_pack(p, 256, 256, 6, 8, p, p, p, p, None, None, p, 1 << 20, None) == UNSUP   # 6:8 with dense_q
    assert L.sbn_quant_act_expand68(None, 4, 256, p, p, None) == NULL
    assert L.sbn_quant_act_expand68(p, 4, 384, p, p, None) == SHAPE
    assert L.sbn_quant_act_expand68(p, 4, 256, odd, p, None) == ALIGN
    assert L.sbn_norm_quant_act_expand68(p, 4, 384, p, ctypes.c_float(1e-6), p, p, None) == SHAPE
    assert L.sbn_norm_quant_act_expand68(p, 4, 16384 + 256, p, ctypes.c_float(1e-6), p, p, None) == UNSUP
    assert L.sbn_norm_quant_act_expand68(p, 4, 256, odd, ctypes.c_float(1e-6), p, p, None) == ALIGN
    assert L.sbn_expanded_k(2560, 6, 8) == 3840 and L.sbn_expanded_k(2560, 2, 4) == 2560
    assert L.sbn_expanded_k(2560 + 128, 6, 8) == 0 and L.sbn_expanded_k(2560, 3, 4) == 0
    assert qmp(N=100) == SHAPE
    assert qmp(K=64) == SHAPE
    assert qmp(wsb=8) == WS
    assert qmp(ws=None) == WS
    assert qmp(prev=p) == NULL           # prev_meta without flip_bits
    assert qmp(W=odd) == ALIGN
    gemm = lambda **k: L.sbn_sparse_bitlinear(k.get("xq", p), p, k.get("T", 64), p, k.get("meta", p), p,
                                              k.get("N", 256), k.get("K", 256), None, p, k.get("dt", 0), None,
                                              k.get("ws"), k.get("wsb", 0), None)
    assert gemm(xq=None) == NULL
    assert gemm(meta=None) == NULL
    assert gemm(T=0) == SHAPE
    assert gemm(N=130) == SHAPE
    assert gemm(K=192) == SHAPE
    assert gemm(dt=5) == UNSUP
    assert gemm(xq=odd) == ALIGN
    L.sbn_set_gemm_tuning(64, 5)                    # split-K through global memory needs its scratch
    try:
        assert gemm(T=4, N=2560, K=2560) == WS
    finally:
        L.sbn_set_gemm_tuning(0, 0)
    assert L.sbn_bitlinear(p, p, 64, None, p, 256, 256, None, p, 0, None, None, 0, None) == NULL
    # packed weights: conversion and the few-token GEMM on them
    assert L.sbn_pack_vals2(None, 256, 256, p, None) == NULL
    assert L.sbn_pack_vals2(p, 100, 256, p, None) == SHAPE
    assert L.sbn_pack_vals2(p, 256, 256, odd, None) == ALIGN
    pk = lambda **k: L.sbn_sparse_bitlinear_packed(k.get("xq", p), p, k.get("T", 16), k.get("v2", p), k.get("meta", p), p,
                                                   k.get("N", 256), k.get("K", 512), None, p, k.get("dt", 0), None, None)
    assert pk(v2=None) == NULL
    assert pk(meta=None) == NULL
    assert pk(T=0) == SHAPE
    assert pk(K=192) == SHAPE
    assert pk(T=2000) == UNSUP              # few tokens only
    assert pk(K=128) == UNSUP               # at least two k-blocks to split
    assert pk(dt=7) == UNSUP
    assert pk(xq=odd) == ALIGN
    from paper_2603_05168_b200 import binding as b
    assert L.sbn_quantize_mask_pack_batched(0, p, p, 1 << 20, None) == SHAPE
    assert L.sbn_quantize_mask_pack_batched(2, None, p, 1 << 20, None) == NULL
    jobs = (b.PackJob * 2)()
    for j in jobs:
        j.W, j.N, j.K, j.vals, j.meta, j.w_scale = 0x1000, 256, 256, 0x1000, 0x1000, 0x1000
    assert L.sbn_quantize_mask_pack_batched(2, ctypes.cast(jobs, ctypes.c_void_p), p, 16, None) == WS
    jobs[1].K = 100
    assert L.sbn_quantize_mask_pack_batched(2, ctypes.cast(jobs, ctypes.c_void_p), p, 1 << 20, None) == SHAPE
    assert b.sbn_batch_workspace_bytes(3) >= 3 * 148 * 16


def test_binding_fails_loudly_without_library(tmp_path, monkeypatch):
    from paper_2603_05168_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError):
        binding.lib()


def test_dispatch_plan_is_sane(L):
    # host-only: the dispatcher's choices for the shapes the benchmarks use (kernel, tile, split, cluster)
    from paper_2603_05168_b200 import binding as b
    assert b.sbn_plan_gemm(True, 4096, 3840, 2560)[0] == 3            # large T, short K: CTA pairs, 256-feature tiles
    assert b.sbn_plan_gemm(True, 8192, 4096, 11008)[0] == 2           # large T, long K: CTA pairs, 512-feature tiles
    k, bn, split, cluster = b.sbn_plan_gemm(True, 16, 3840, 2560)     # few tokens: cluster split-K, 32-token tile
    assert (k, bn, split) == (1, 32, 1) and cluster in (2, 3, 4)
    for T in (1, 16, 32):
        for (N, K) in ((3840, 2560), (2560, 6912), (11008, 4096), (4096, 11008)):
            k, bn, split, cluster = b.sbn_plan_gemm(True, T, N, K)
            assert k == 1 and split == 1 and cluster in (2, 3, 4), (T, N, K)
            tiles = (N // 128) * ((T + bn - 1) // bn)
            assert tiles * cluster <= (296 if bn <= 64 else 148)       # every CTA resident at once
    assert b.sbn_plan_gemm(True, 16, 100, 2560) == (0, 0, 0, 0)        # illegal shape


def test_fused_entry_validation_on_host(L):
    p = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1004)
    NULL, SHAPE, ALIGN, UNSUP = 1, 2, 3, 4
    fs = lambda **k: L.sbn_quant_act_sparse_bitlinear(k.get("x", p), k.get("T", 8), p, k.get("meta", p), p, k.get("N", 256),
                                                      k.get("K", 512), None, p, k.get("dt", 0), None, None, None)
    assert fs(x=None) == NULL
    assert fs(meta=None) == NULL
    assert fs(T=0) == SHAPE
    assert fs(N=100) == SHAPE
    assert fs(T=300) == UNSUP
    assert fs(K=128) == UNSUP
    assert fs(dt=9) == UNSUP
    assert fs(x=odd) == ALIGN
    assert L.sbn_quant_act_bitlinear(p, 8, None, p, 256, 512, None, p, 0, None, None, None) == NULL


def test_canonical_layout_calls_validate_on_host(L):
    p, q = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x2000)
    odd = ctypes.c_void_p(0x1008)
    NULL, SHAPE, ALIGN, UNSUP = 1, 2, 3, 4
    for fn in (L.sbn_unpack_canonical, L.sbn_tile_canonical):
        assert fn(None, None, 256, 256, None, None, None) == NULL          # nothing to convert
        assert fn(p, None, 256, 256, None, None, None) == NULL             # a source without its destination
        assert fn(p, p, 256, 100, q, q, None) == SHAPE
        assert fn(p, p, 0, 256, q, q, None) == SHAPE
        assert fn(odd, p, 256, 256, q, q, None) == ALIGN
        assert fn(p, p, 256, 256, p, q, None) == UNSUP                     # in place
