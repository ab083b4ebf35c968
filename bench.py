#!/usr/bin/env python
"""Benchmark of the 2:4-sparse ternary BitLinear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" = one pass of the whole path over the four BitNet-2B-shaped BitLinears at T = 4096
tokens: for every layer  quantize/mask/pack(W fp32)  ->  quant_act(x bf16)  ->  sparse BitLinear
(bf16 output).  Rank 0 prints ONE JSON line.  `value` is dense-equivalent tera-ops per second of
the whole step (2*T*N*K summed over the four GEMMs, divided by the step time, summed over GPUs);
the per-kernel and per-shape numbers that explain it ride along in the same line.

Multi-GPU: the path has no exchange step, so N GPUs run N independent replicas ("replicas only",
weak scaling); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_05168_b200 import inputs  # noqa: E402

# NVIDIA's HGX B200 datasheet figures per GPU (dense; the sparse figure is twice that).
DATASHEET_INT8_DENSE_TOPS = 4500.0
DATASHEET_INT8_SPARSE_TOPS = 9000.0
NOMINAL_BF16_DENSE_TFLOPS = 2250.0
# dram__bytes_read.sum + dram__bytes_write.sum of the sparse GEMM per launch come from the ncu captures
# summarised under profiles/ (the outputs mostly stay in L2, so this is far below the algorithmic operand
# + output bytes -- the kernel is tensor-bound, the figure is context).
GEMM_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "gemm_dram_traffic.json")
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0

T_TOKENS = 4096
# name -> (tokens, [(layer, K, N)], weight sigma, outlier prob, per-token lognormal sigma)
WORKLOADS = {
    "2b": (4096, inputs.SHAPES_2B, 0.02, 0.0, 0.0),
    "7b": (8192, inputs.SHAPES_7B, 0.015, 0.05, 0.5),
    "down7b": (8192, inputs.SHAPES_7B[1:], 0.015, 0.05, 0.5),      # one layer: small case for profiling
}
METRIC = "2:4 sparse ternary BitLinear TOPS, % sparse-INT8 peak, speedup vs dense ternary"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS,
                bf16_tflops_sustained=1400.0, source="fallback")


def gemm_dram_traffic(workload):
    """Measured DRAM bytes per sparse-GEMM launch of this workload's step (None if no capture is on file)."""
    try:
        with open(GEMM_TRAFFIC_FILE) as f:
            return float(json.load(f)[workload]["bytes_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


def workload_string(name, T, shapes):
    return (f"{name}: BitLinears at T={T}: " + ", ".join(f"{n} {K}->{N}" for n, K, N in shapes) +
            "; step = quantize_mask_pack of all layers (one batched launch, previous step's scales as hints), then quant_act + sparse_bitlinear (bf16 out) per layer")


def max_over_ranks(ms_local, world, dist=None, device="cpu"):
    """Replicas only: every rank runs the same work on its own GPU, nothing is exchanged on the data
    path; the job's step time is the slowest rank's device time."""
    if world <= 1:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_replica, world, ms_per_step):
    """Units processed by all ranks divided by the (max over ranks) step time."""
    return ops_per_replica * world / (ms_per_step * 1e-3) / 1e12


def step_ops(T, shapes=inputs.SHAPES_2B):
    return sum(2.0 * T * N * K for _, K, N in shapes)


# ------------------------------------------------------------------------------------------------
# clocks sampled during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.thread = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._reader, daemon=True)
        self.thread.start()

    def _reader(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0, t1):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for (ts, r) in self.rows if t0 - 0.05 <= ts <= t1 + 0.15] or [r for (_, r) in self.rows]
        for r in rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_mhz_min": min(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_step(sample_tokens: int, cache: dict):
    """One pass of the path through the CPU oracle on `sample_tokens` tokens of every layer.
    Returns seconds."""
    import oracle
    if "data" not in cache:
        cache["data"] = [(inputs.latent_weights(N, K, seed=1 + i),
                          inputs.activations_bf16(sample_tokens, K, seed=11 + i))
                         for i, (_, K, N) in enumerate(inputs.SHAPES_2B)]
    t0 = time.perf_counter()
    for W, x in cache["data"]:
        r = oracle.quantize_mask_pack(W)
        xq, s = oracle.quant_act(x)
        y, _ = oracle.sparse_bitlinear(xq, s, r["vals"], r["meta"], r["scale"])
        oracle.f32_to_bf16_bits(y)
    return time.perf_counter() - t0


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only), on the very
    workload the GPU arm times: all T = 4096 tokens of all four layers per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    sample = T_TOKENS
    cache = {}
    for _ in range(args.warmup):
        oracle_step(sample, cache)
    times = [oracle_step(sample, cache) for _ in range(args.steps)]
    total = sum(times)
    value = step_ops(sample) * args.steps / total / 1e12
    cores = oracle.num_threads()
    in_bytes = sum(N * K * 4 + sample * K * 2 for _, K, N in inputs.SHAPES_2B)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic",
        "config": {"workload": workload_string("2b", sample, inputs.SHAPES_2B), "tokens": sample, "parallelism": "single",
                   "l2": f"step streams {in_bytes / 1e6:.0f} MB of inputs (host arm: the CPU oracle on the host cores)"},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": cores, "kind": "oracle",
                         "sample": f"all {sample} tokens per layer, all four weight matrices in full, every step"},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
class Layer:
    """Device (and pinned host) buffers of one BitLinear of the workload."""

    def __init__(self, name, K, N, T, seed, torch, b, sigma=0.02, outl=0.0, logn=0.0, masters="fp32"):
        self.name, self.K, self.N, self.T = name, K, N, T
        W = inputs.latent_weights(N, K, seed=seed, sigma=sigma, outlier_prob=outl)
        x = inputs.activations_bf16(T, K, seed=seed + 10, token_lognormal_sigma=logn)
        if masters == "bf16":     # master weights kept in bf16 (the paper's own example)
            self.W_host = torch.from_numpy(inputs.f32_to_bf16_bits(W).view(np.int16)).view(torch.bfloat16).pin_memory()
        else:
            self.W_host = torch.from_numpy(W).pin_memory()
        self.w_bytes = self.W_host.element_size()
        self.x_host = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory()
        self.W = self.W_host.cuda()
        self.x = self.x_host.cuda()
        self.W_stage = torch.empty_like(self.W)
        self.x_stage = torch.empty_like(self.x)
        self.packed = b.alloc_packed(N, K, with_dense=True)
        self.xq = b.alloc_xq(T, K)
        self.a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
        self.gain = torch.from_numpy((1.0 + 0.1 * np.random.default_rng(seed + 20).standard_normal(K)).astype(np.float32)).cuda()
        self.y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        self.y32 = torch.empty((T, N), dtype=torch.float32, device="cuda")
        self.y_host = torch.empty((T, N), dtype=torch.bfloat16).pin_memory()
        self.ws = b.alloc_gemm_ws(b.OP_SPARSE_BITLINEAR, T, N, K)
        self.ops = 2.0 * T * N * K


def backward_rows(torch, b, peaks, layers, time_cold, iters):
    """The layer's backward under the dual straight-through estimator (Sec. 2.3, Eq. 5): dX = dY w_masked and
    the dense dW = dY^T x_q on the tensor cores in bf16 (fp32 accumulation), per 2B-shaped layer at
    T = 4096, cold L2.  Each time covers the whole call for that gradient: the operand preparation (W_eff^T,
    or x_q, in bf16) and the GEMM; `both_us` is one call for both gradients (the two GEMMs share the machine
    where the first one's last wave leaves pairs idle).  `library_matmul_*`: torch.matmul on ready-made bf16 operands of
    the same shapes, as the pace of a library GEMM on this machine (context, not part of the path)."""
    rows = {}
    for L in layers:
        T, N, K = L.T, L.N, L.K
        p = L.packed
        b.sbn_quantize_mask_pack(L.W, p["vals"], p["meta"], p["w_scale"], p["ws"])
        b.sbn_quant_act(L.x, L.xq, L.a_scale)
        dY = torch.from_numpy(inputs.activations_bf16(T, N, seed=77).view(np.int16)).cuda().view(torch.bfloat16)
        dX = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
        dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
        ws = torch.empty(b.sbn_workspace_bytes(b.OP_BACKWARD, T, N, K), dtype=torch.uint8, device="cuda")
        f_dx = lambda: b.sbn_bitlinear_backward(dY, L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], N, K, dX=dX, ws=ws)
        f_dw = lambda: b.sbn_bitlinear_backward(dY, L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], N, K, dW=dW, ws=ws)
        f_both = lambda: b.sbn_bitlinear_backward(dY, L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], N, K, dX=dX, dW=dW, ws=ws)
        w_b = torch.empty((N, K), dtype=torch.bfloat16, device="cuda").normal_()
        g_dx = lambda: torch.matmul(dY, w_b)
        g_dw = lambda: torch.matmul(dY.t(), L.x)
        for fn in (f_dx, f_dw, f_both, g_dx, g_dw):
            for _ in range(2):
                fn()
        t = {k: time_cold(fn, iters) for k, fn in (("dx", f_dx), ("dw", f_dw), ("both", f_both), ("lib_dx", g_dx), ("lib_dw", g_dw))}
        flops = 2.0 * T * N * K
        rows[L.name] = {"dx_us": round(t["dx"], 2), "dw_us": round(t["dw"], 2),
                        "both_us": round(t["both"], 2), "both_tflops": round(2.0 * flops / t["both"] / 1e6, 1),
                        "dx_tflops": round(flops / t["dx"] / 1e6, 1), "dw_tflops": round(flops / t["dw"] / 1e6, 1),
                        "dx_frac_of_measured_bf16_burst": round(flops / t["dx"] / 1e6 / peaks["bf16_tflops"], 4),
                        "dw_frac_of_measured_bf16_burst": round(flops / t["dw"] / 1e6 / peaks["bf16_tflops"], 4),
                        "library_matmul_dx_us": round(t["lib_dx"], 2), "library_matmul_dw_us": round(t["lib_dw"], 2)}
        del dY, dX, dW, ws, w_b
    b.sbn_check_status()
    return rows


def large_m_and_sustained(torch, b, peaks, sampler, time_cold, iters):
    """The large-M target on the two 7B-class shapes (T = 8192; weights N(0, 0.015) with 5 % x10 outliers,
    activations with a per-token LogNormal(0, 0.5) scale): isolated sparse and dense GEMM, cold L2, both
    output dtypes; then the down projection's GEMM launched back to back for >= 2 s (sparse, then dense)
    with the SM clock sampled meanwhile -- what the kernel sustains, next to the burst figure."""
    stream = torch.cuda.current_stream()
    rows, sustained = {}, {}
    ratio = DATASHEET_INT8_SPARSE_TOPS / NOMINAL_BF16_DENSE_TFLOPS
    for i, (name, K, N) in enumerate(inputs.SHAPES_7B):
        T = 8192
        W = torch.from_numpy(inputs.latent_weights(N, K, seed=1 + i, sigma=0.015, outlier_prob=0.05)).cuda()
        x = torch.from_numpy(inputs.activations_bf16(T, K, seed=11 + i, token_lognormal_sigma=0.5).view(np.int16)).cuda().view(torch.bfloat16)
        p = b.alloc_packed(N, K, with_dense=True)
        b.sbn_quantize_mask_pack(W, p["vals"], p["meta"], p["w_scale"], p["ws"], dense_q=p["dense_q"])
        del W
        xq = b.alloc_xq(T, K)
        a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
        b.sbn_quant_act(x, xq, a_scale)
        del x
        ops = 2.0 * T * N * K
        row = {"T": T, "K": K, "N": N}
        ys = {"bf16": torch.empty((T, N), dtype=torch.bfloat16, device="cuda"), "f32": torch.empty((T, N), dtype=torch.float32, device="cuda")}
        sp_fn = lambda y: b.sbn_sparse_bitlinear(xq, a_scale, p["vals"], p["meta"], p["w_scale"], y)
        de_fn = lambda y: b.sbn_bitlinear(xq, a_scale, p["dense_q"], p["w_scale"], y)
        for tag, y in ys.items():
            for _ in range(3):
                sp_fn(y)
                de_fn(y)
            sp = time_cold(lambda: sp_fn(y), iters)
            de = time_cold(lambda: de_fn(y), iters)
            row[tag] = {"sparse_us": round(sp, 2), "dense_us": round(de, 2),
                        "sparse_tops": round(ops / sp / 1e6, 1), "dense_tops": round(ops / de / 1e6, 1),
                        "pct_sparse_int8_datasheet": round(100 * ops / sp / 1e6 / DATASHEET_INT8_SPARSE_TOPS, 1),
                        "pct_of_measured_bf16_burst_x4": round(100 * ops / sp / 1e6 / (peaks["bf16_tflops"] * ratio), 1),
                        "speedup_vs_dense": round(de / sp, 3)}
        rows[name] = row
        if name == "down_7b":
            y = ys["bf16"]
            for tag, fn in (("sparse", sp_fn), ("dense", de_fn)):
                fn(y)
                torch.cuda.synchronize()
                a = torch.cuda.Event(enable_timing=True)
                c = torch.cuda.Event(enable_timing=True)
                t0 = time.time()
                a.record(stream)
                n = 0
                while time.time() - t0 < 2.2:                      # the queue fills, then the host enqueues at the GPU's pace
                    for _ in range(64):
                        fn(y)
                    n += 64
                c.record(stream)
                torch.cuda.synchronize()
                t1 = time.time()
                ms = a.elapsed_time(c)
                clk = sampler.summary(t0 + 0.3, t1 - 0.05)            # samples well inside the loaded interval
                tops = ops * n / (ms * 1e-3) / 1e12
                peak_sus = peaks["bf16_tflops_sustained"] * (ratio if tag == "sparse" else ratio / 2)
                sm = clk["sm_mhz"]
                sustained[tag] = {"launches": n, "seconds": round(ms * 1e-3, 3), "us_per_launch": round(ms * 1e3 / n, 2), "tops": round(tops, 1),
                                  "pct_int8_datasheet": round(100 * tops / (DATASHEET_INT8_SPARSE_TOPS if tag == "sparse" else DATASHEET_INT8_DENSE_TOPS), 1),
                                  "frac_of_measured_bf16_sustained_x_ratio": round(tops / peak_sus, 4),
                                  "sm_mhz_median": sm, "sm_mhz_min": clk.get("sm_mhz_min"), "sm_max_mhz": clk["sm_max_mhz"],
                                  "reasons": clk["reasons"], "clock_samples": clk["samples"],
                                  "tops_scaled_to_max_clock": round(tops * clk["sm_max_mhz"] / sm, 1) if sm else None}
            sustained["workload"] = f"down_7b {K}->{N} at T={T}, bf16 out, same launch back to back for >= 2 s (L2-warm)"
            sustained["peak_source"] = (f"{peaks['source']} bf16 sustained {peaks['bf16_tflops_sustained']} TFLOP/s x {ratio:g} (sparse int8) "
                                        f"or x {ratio / 2:g} (dense int8), nominal ratios")
        del p, xq, ys
        torch.cuda.empty_cache()
    return rows, sustained


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        sbn_build.build()
    if world > 1:
        dist.barrier()
    b.lib()
    peaks = load_peaks()
    T, shapes, sigma, outl, logn = WORKLOADS[args.workload]
    layers = [Layer(n, K, N, T, seed=1 + i, torch=torch, b=b, sigma=sigma, outl=outl, logn=logn, masters=args.masters)
              for i, (n, K, N) in enumerate(shapes)]
    in_bytes = sum(L.W.numel() * L.w_bytes + L.x.numel() * 2 for L in layers)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    KERNELS = ("quantize_mask_pack", "quant_act", "sparse_bitlinear")

    # One launch re-quantises, masks and packs all layers' weights (the batched entry point runs
    # pass 1 of matrix m + 1 under the exchange and pass 2 of matrix m); then, per layer, the
    # activation quantiser and the sparse GEMM.
    # gamma_hint = the scale the previous step left in w_scale (a dynamic-mask training step re-packs
    # slowly drifting weights): the kernel then need not sample the matrix before it streams it.
    pack_jobs = b.make_pack_jobs([dict(W=L.W, vals=L.packed["vals"], meta=L.packed["meta"], w_scale=L.packed["w_scale"],
                                       gamma_hint=L.packed["w_scale"])
                                  for L in layers])
    pack_ws = torch.empty(b.sbn_batch_workspace_bytes(len(layers)), dtype=torch.uint8, device="cuda")

    def step(evs=None):
        ev = lambda: torch.cuda.Event(enable_timing=True)
        if evs is not None:
            e0, e1 = ev(), ev()
            e0.record(stream)
        b.sbn_quantize_mask_pack_batched(pack_jobs, pack_ws)
        if evs is not None:
            e1.record(stream)
            evs.append(("quantize_mask_pack", "all_layers_batched", e0, e1))
        for L in layers:
            p = L.packed
            if evs is not None:
                e = [ev() for _ in range(3)]
                e[0].record(stream)
            b.sbn_quant_act(L.x, L.xq, L.a_scale)
            if evs is not None:
                e[1].record(stream)
            b.sbn_sparse_bitlinear(L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], L.y, ws=L.ws)
            if evs is not None:
                e[2].record(stream)
                evs.append(("quant_act", L.name, e[0], e[1]))
                evs.append(("sparse_bitlinear", L.name, e[1], e[2]))

    # ---- device-resident timing -----------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    b.sbn_check_status()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    evs = []
    barrier()
    launches0 = b.sbn_launch_count()
    t_wall0 = time.time()
    # The kernels are short (tens of microseconds), so the timed region must not depend on how
    # fast the host can enqueue them: the steps are enqueued in chunks behind a device-side delay
    # (outside the timed region) that lets the host run ahead; every chunk is timed by its own
    # pair of events on the launching stream and the times are added up -- exactly K steps.
    chunk_times = []
    done = 0
    while done < args.steps:
        n_chunk = min(8, args.steps - done)
        a_ev = torch.cuda.Event(enable_timing=True)
        c_ev = torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(6e6 + n_chunk * 2.5e6))
        a_ev.record(stream)
        for _ in range(n_chunk):
            step()
        c_ev.record(stream)
        chunk_times.append((a_ev, c_ev))
        done += n_chunk
        torch.cuda.synchronize()
    barrier()
    t_wall1 = time.time()
    launches = b.sbn_launch_count() - launches0
    b.sbn_check_status()
    ms_total = sum(a_ev.elapsed_time(c_ev) for a_ev, c_ev in chunk_times)
    ms_total = max_over_ranks(ms_total, world, dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = whole_job_tops(step_ops(T, shapes), world, ms_per_step)

    # per-kernel times inside the step sequence: a separate, instrumented pass (an event between
    # two kernels would keep the second from starting its prologue under the first one's tail)
    torch.cuda._sleep(int(6e6))
    for _ in range(min(args.steps, 8)):
        step(evs)
    torch.cuda.synchronize()
    per_kernel = {k: {} for k in KERNELS}
    for k, name, ea, eb in evs:
        per_kernel[k].setdefault(name, []).append(ea.elapsed_time(eb) * 1e3)   # us
    kernel_us = {k: {n: statistics.mean(v) for n, v in d.items()} for k, d in per_kernel.items()}

    if args.only_step:
        sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": "TOPS", "ms_per_step": ms_per_step,
                              "workload": args.workload, "gpu_launches": int(launches),
                              "kernel_us_in_step": {k: {n: round(v, 2) for n, v in d.items()} for k, d in kernel_us.items()}}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end-to-end: host buffers, copies inside the timed region ----------------------------------
    # Layers alternate between two streams, so the device-to-host copy of one layer's y runs while
    # the next layer's W and x come in (the link is full duplex); each layer has its own staging
    # buffers, and a layer always uses the same stream, which orders its reuse across steps.
    e2e_streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    # The pack kernel's CTAs exchange partial sums, so two pack calls must never overlap on the GPU (see
    # sbn.h): all of them go to one stream of their own, each behind the copy of its W, and a layer's
    # forward waits for its pack.
    pack_stream = torch.cuda.Stream()

    def e2e_step():
        for i, L in enumerate(layers):
            p = L.packed
            st = e2e_streams[i % 2]
            with torch.cuda.stream(st):
                L.W_stage.copy_(L.W_host, non_blocking=True)
                w_in = torch.cuda.Event()
                w_in.record(st)
            with torch.cuda.stream(pack_stream):
                pack_stream.wait_event(w_in)
                b.sbn_quantize_mask_pack(L.W_stage, p["vals"], p["meta"], p["w_scale"], p["ws"])
                packed = torch.cuda.Event()
                packed.record(pack_stream)
            with torch.cuda.stream(st):
                st.wait_event(packed)
                b.sbn_layer_forward_host(L.x_host, L.x_stage, L.xq, L.a_scale, p["w_scale"], L.y, L.y_host,
                                         vals=p["vals"], meta=p["meta"], ws=L.ws)
    e2e_steps = max(2, min(args.steps, 5))
    for _ in range(2):
        e2e_step()
    barrier()
    s2 = torch.cuda.Event(enable_timing=True)
    e2 = torch.cuda.Event(enable_timing=True)
    s2.record(stream)
    for st in e2e_streams + [pack_stream]:
        st.wait_event(s2)
    for _ in range(e2e_steps):
        e2e_step()
    for st in e2e_streams + [pack_stream]:
        done_ev = torch.cuda.Event()
        done_ev.record(st)
        stream.wait_event(done_ev)
    e2.record(stream)
    barrier()
    b.sbn_check_status()
    e2e_ms = max_over_ranks(s2.elapsed_time(e2), world, dist, "cuda") / e2e_steps
    e2e_value = whole_job_tops(step_ops(T, shapes), world, e2e_ms)
    h2d = sum(L.W_host.numel() * L.w_bytes + L.x_host.numel() * 2 for L in layers)
    d2h = sum(L.y_host.numel() * 2 for L in layers)

    # ---- isolated kernels, cold L2 (a 512 MB buffer is overwritten before every launch) --------
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    def time_cold(fn, iters):
        evp = []
        torch.cuda._sleep(int(4e6 + iters * 1e6))          # host runs ahead; the flush also covers gaps
        for _ in range(iters):
            flush.zero_()
            a = torch.cuda.Event(enable_timing=True)
            c = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            c.record(stream)
            evp.append((a, c))
        torch.cuda.synchronize()
        ts = sorted(a.elapsed_time(c) * 1e3 for a, c in evp)
        return statistics.median(ts)

    iters = 12
    gemm = {}
    for L in layers:
        p = L.packed
        b.sbn_quantize_mask_pack(L.W, p["vals"], p["meta"], p["w_scale"], p["ws"], dense_q=p["dense_q"])
        b.sbn_quant_act(L.x, L.xq, L.a_scale)
        row = {}
        for tag, y in (("bf16", L.y), ("f32", L.y32)):
            for _ in range(3):
                b.sbn_sparse_bitlinear(L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], y, ws=L.ws)
                b.sbn_bitlinear(L.xq, L.a_scale, p["dense_q"], p["w_scale"], y, ws=L.ws)
            sp = time_cold(lambda: b.sbn_sparse_bitlinear(L.xq, L.a_scale, p["vals"], p["meta"], p["w_scale"], y, ws=L.ws), iters)
            de = time_cold(lambda: b.sbn_bitlinear(L.xq, L.a_scale, p["dense_q"], p["w_scale"], y, ws=L.ws), iters)
            row[tag] = {"sparse_us": round(sp, 2), "dense_us": round(de, 2),
                        "sparse_tops": round(L.ops / sp / 1e6, 1), "dense_tops": round(L.ops / de / 1e6, 1),
                        "pct_sparse_int8_datasheet": round(100 * L.ops / sp / 1e6 / DATASHEET_INT8_SPARSE_TOPS, 1),
                        "speedup_vs_dense": round(de / sp, 3)}
        qmp = time_cold(lambda: b.sbn_quantize_mask_pack(L.W, p["vals"], p["meta"], p["w_scale"], p["ws"]), iters)
        act = time_cold(lambda: b.sbn_quant_act(L.x, L.xq, L.a_scale), iters)
        row["quantize_mask_pack_us"] = round(qmp, 2)
        row["quantize_mask_pack_gbs"] = round(L.N * L.K * (L.w_bytes + 0.625) / qmp / 1e3, 1)     # algorithmic bytes: W once + vals + meta
        # the same matrix as a batch of one whose job carries the previous scale as its estimate of gamma (what a
        # training loop does: no sample, a narrow bracket)
        hint_jobs = b.make_pack_jobs([dict(W=L.W, vals=p["vals"], meta=p["meta"], w_scale=p["w_scale"], gamma_hint=p["w_scale"])])
        hint_ws = torch.empty(b.sbn_batch_workspace_bytes(1), dtype=torch.uint8, device="cuda")
        b.sbn_quantize_mask_pack_batched(hint_jobs, hint_ws)
        qmp_h = time_cold(lambda: b.sbn_quantize_mask_pack_batched(hint_jobs, hint_ws), iters)
        row["quantize_mask_pack_hint_us"] = round(qmp_h, 2)
        row["quantize_mask_pack_hint_gbs"] = round(L.N * L.K * (L.w_bytes + 0.625) / qmp_h / 1e3, 1)
        row["quant_act_us"] = round(act, 2)
        row["quant_act_gbs"] = round((L.T * L.K * 3 + L.T * 4) / act / 1e3, 1)
        # the same kernel launched back to back over 8 distinct inputs (more than the L2 holds): what a
        # launch costs inside a stream of kernels, without the ~6 us an isolated launch spends between two events
        xs = [L.x] + [torch.empty_like(L.x).copy_(L.x) for _ in range(7)]
        torch.cuda.synchronize()
        torch.cuda._sleep(int(4e6))
        ea, ec = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ea.record(stream)
        for r_i in range(32):
            b.sbn_quant_act(xs[r_i % 8], L.xq, L.a_scale)
        ec.record(stream)
        torch.cuda.synchronize()
        act_st = ea.elapsed_time(ec) * 1e3 / 32
        del xs
        row["quant_act_stream_us"] = round(act_st, 2)
        row["quant_act_stream_gbs"] = round((L.T * L.K * 3 + L.T * 4) / act_st / 1e3, 1)
        row["quant_act_stream_frac_of_hbm"] = round((L.T * L.K * 3 + L.T * 4) / act_st / 1e3 / peaks["hbm_gbs"], 4)
        if L.K <= 16384:
            # Algorithm 1's x~ = Q_a(Norm(x)) as one kernel (RMSNorm with gain fused into the quantiser)
            nact = time_cold(lambda: b.sbn_norm_quant_act(L.x, L.xq, L.a_scale, gain=L.gain, eps=1e-6), iters)
            row["norm_quant_act_us"] = round(nact, 2)
            row["norm_quant_act_gbs"] = round((L.T * L.K * 3 + L.T * 4 + L.K * 4) / nact / 1e3, 1)
        gemm[L.name] = row
    b.sbn_check_status()
    large_m, sustained, few_tokens, backward = None, None, None, None
    if rank == 0 and world == 1 and args.workload == "2b" and not args.no_extras:
        backward = backward_rows(torch, b, peaks, layers, time_cold, iters)
        large_m, sustained = large_m_and_sustained(torch, b, peaks, sampler, time_cold, iters)
        few_tokens = decode_rows(torch, b, peaks, inputs.SHAPES_2B, (1, 4, 16, 64), cold=False)
        b.sbn_check_status()
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)

    # ---- roofline of the dominant kernel of the step -------------------------------------------------
    tot = {k: sum(v.values()) for k, v in kernel_us.items()}
    dominant = max(tot, key=tot.get)
    if dominant == "sparse_bitlinear":
        # a real contraction: sparse int8 tensor pipe.  Peak = measured bf16 burst x the nominal
        # sparse-int8 : dense-bf16 ratio (4x).
        ratio = DATASHEET_INT8_SPARSE_TOPS / NOMINAL_BF16_DENSE_TFLOPS
        peak = peaks["bf16_tflops"] * ratio
        achieved = sum(L.ops for L in layers) / (tot[dominant] * 1e-6) / 1e12
        roofline = {"bound": "tensor", "kernel": "bitlinear_gemm_pair_kernel<sparse, 1>" if args.workload == "2b" else "bitlinear_gemm_pair_kernel<sparse, 2>", "achieved": round(achieved, 1),
                    "peak": round(peak, 1), "unit": "TOP/s", "frac": round(achieved / peak, 4),
                    "traffic": gemm_dram_traffic(args.workload),
                    "traffic_source": "profiles/gemm_dram_traffic.json (ncu capture of this step)",
                    "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TFLOP/s x {ratio:g} (nominal sparse-int8 : bf16)",
                    "frac_of_datasheet_sparse_int8": round(achieved / DATASHEET_INT8_SPARSE_TOPS, 4)}
    else:
        per_param = (layers[0].w_bytes + 0.625) if dominant == "quantize_mask_pack" else None
        if dominant == "quantize_mask_pack":
            bytes_ = sum(L.N * L.K * per_param for L in layers)
        else:
            bytes_ = sum(L.T * L.K * 3 + L.T * 4 for L in layers)
        achieved = bytes_ / (tot[dominant] * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4), "traffic": None,
                    "peak_source": peaks["source"]}

    # ---- CPU oracle baseline (rank 0, single GPU runs only) --------------------------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.workload == "2b":
        import oracle
        sample, passes = T, 2                           # about 10-20 s of host time on 16 cores
        cache = {}
        secs = sum(oracle_step(sample, cache) for _ in range(passes))
        cpu_baseline = {"value": step_ops(sample) * passes / secs / 1e12, "unit": "TOPS", "cores": oracle.num_threads(),
                        "kind": "oracle", "seconds": round(secs, 2),
                        "sample": f"all {sample} tokens per layer, all four weight matrices in full, {passes} passes"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": workload_string(args.workload, T, shapes),
                       "tokens": T, "parallelism": "replicas" if world > 1 else "single",
                       "l2": f"step streams {in_bytes / 1e6:.0f} MB of inputs (> 126 MB L2); isolated-kernel numbers flush L2 before every launch"},
            "e2e": {"value": e2e_value, "unit": "TOPS", "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "cpu_baseline": cpu_baseline,
            "kernel_us_in_step": {k: {n: round(v, 2) for n, v in d.items()} for k, d in kernel_us.items()},
            "isolated": gemm,
            "backward": backward,
            "isolated_large_m": large_m,
            "sustained": sustained,
            "few_tokens": few_tokens,
            "datasheet_int8_tops": {"dense": DATASHEET_INT8_DENSE_TOPS, "sparse": DATASHEET_INT8_SPARSE_TOPS},
            "measured_peaks": peaks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()



# ------------------------------------------------------------------------------------------------
# Secondary workloads (each prints its own JSON line; the headline line is run_ours)
# ------------------------------------------------------------------------------------------------
def _cold_timer(torch, stream, flush):
    def time_cold(fn, iters):
        evp = []
        torch.cuda._sleep(int(4e6 + iters * 1e6))
        for _ in range(iters):
            flush.zero_()
            a = torch.cuda.Event(enable_timing=True)
            c = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            c.record(stream)
            evp.append((a, c))
        torch.cuda.synchronize()
        return statistics.median(sorted(a.elapsed_time(c) * 1e3 for a, c in evp))
    return time_cold


def decode_rows(torch, b, peaks, shapes, token_counts, big=False, cold=True):
    """Few-token rows: for every (matrix, T) the sparse and the dense BitLinear, `stream` = launches back
    to back over enough distinct weight copies that every launch reads its weights from HBM (what a
    decode loop over the layers of a model sees), and optionally `cold` = one launch after 512 MB were
    written over L2 (includes the ~6 us an empty launch costs between two events).  Memory-bound: GB/s of
    algorithmic bytes (weights + activations + outputs) against the measured HBM rate."""
    stream = torch.cuda.current_stream()
    time_cold = None
    if cold:
        flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        time_cold = _cold_timer(torch, stream, flush)

    def time_stream(fns, reps=48):
        for f in fns:
            f()
        torch.cuda.synchronize()
        torch.cuda._sleep(int(8e6))
        a = torch.cuda.Event(enable_timing=True)
        c = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for r in range(reps):
            fns[r % len(fns)]()
        c.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(c) * 1e3 / reps

    rows = []
    for i, (name, K, N) in enumerate(shapes):
        W = torch.from_numpy(inputs.latent_weights(N, K, seed=1 + i)).cuda()
        n_copies = min(24, int(200e6 // (N * K * 0.625)) + 1)        # > L2 worth of compressed weights
        packs = []
        for c in range(n_copies):
            p = b.alloc_packed(N, K, with_dense=True)
            b.sbn_quantize_mask_pack(W, p["vals"], p["meta"], p["w_scale"], p["ws"], dense_q=p["dense_q"])
            if big:                                                 # values at two bits each next to the metadata
                p["vals2"] = b.alloc_vals2(N, K)
                b.sbn_pack_vals2(p["vals"], p["vals2"])
            packs.append(p)
            W.mul_(-1.0)                                            # another matrix, same statistics
        p = packs[0]
        for T in token_counts:
            x = torch.from_numpy(inputs.activations_bf16(T, K, seed=50 + T).view(np.int16)).cuda().view(torch.bfloat16)
            xq = b.alloc_xq(T, K)
            a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
            y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
            ws_s = b.alloc_gemm_ws(b.OP_SPARSE_BITLINEAR, T, N, K)
            ws_d = b.alloc_gemm_ws(b.OP_BITLINEAR, T, N, K)
            b.sbn_quant_act(x, xq, a_scale)
            for _ in range(3):
                b.sbn_sparse_bitlinear(xq, a_scale, p["vals"], p["meta"], p["w_scale"], y, ws=ws_s)
                b.sbn_bitlinear(xq, a_scale, p["dense_q"], p["w_scale"], y, ws=ws_d)
            io = T * K + T * N * 2 + T * 4
            sp_bytes = N * K * 0.625 + io
            de_bytes = N * K * 1.0 + io
            row = {"layer": name, "T": T}
            if cold:
                sp = time_cold(lambda: b.sbn_sparse_bitlinear(xq, a_scale, p["vals"], p["meta"], p["w_scale"], y, ws=ws_s), 15)
                de = time_cold(lambda: b.sbn_bitlinear(xq, a_scale, p["dense_q"], p["w_scale"], y, ws=ws_d), 15)
                row.update({"sparse_us": round(sp, 2), "dense_us": round(de, 2),
                            "sparse_gbs": round(sp_bytes / sp / 1e3, 1), "dense_gbs": round(de_bytes / de / 1e3, 1),
                            "speedup_vs_dense": round(de / sp, 3),
                            "sparse_frac_of_hbm": round(sp_bytes / sp / 1e3 / peaks["hbm_gbs"], 4)})
            sp_st = time_stream([(lambda q=q: b.sbn_sparse_bitlinear(xq, a_scale, q["vals"], q["meta"], q["w_scale"], y, ws=ws_s))
                                 for q in packs])
            de_st = time_stream([(lambda q=q: b.sbn_bitlinear(xq, a_scale, q["dense_q"], q["w_scale"], y, ws=ws_d))
                                 for q in packs])
            if big:
                pk_st = time_stream([(lambda q=q: b.sbn_sparse_bitlinear_packed(xq, a_scale, q["vals2"], q["meta"], q["w_scale"], y))
                                     for q in packs])
                row.update({"packed_stream_us": round(pk_st, 2), "packed_stream_gbs": round((N * K * 0.25 + io) / pk_st / 1e3, 1),
                            "packed_vs_int8_held": round(sp_st / pk_st, 3)})
            row.update({"sparse_stream_us": round(sp_st, 2), "dense_stream_us": round(de_st, 2),
                        "sparse_stream_gbs": round(sp_bytes / sp_st / 1e3, 1), "dense_stream_gbs": round(de_bytes / de_st / 1e3, 1),
                        "stream_speedup_vs_dense": round(de_st / sp_st, 3),
                        "sparse_stream_frac_of_hbm": round(sp_bytes / sp_st / 1e3 / peaks["hbm_gbs"], 4)})
            rows.append(row)
        del packs
    return rows


def run_decode_sweep(args):
    """Small-T regime (the paper's decode table is M = 64..512): T in {1, 4, 16, 64, 128, 256, 512} over
    the four 2B-shaped matrices (decode7b: T <= 64 over 7B-class matrices, with the 2-bit packed
    weights as a third arm), sparse vs dense, cold and streamed (see decode_rows)."""
    import torch
    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build
    sbn_build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    peaks = load_peaks()
    big = args.workload == "decode7b"
    shapes = [("gate_up_7b", 4096, 11008), ("down_7b", 11008, 4096), ("qkv_7b", 4096, 12288), ("o_7b", 4096, 4096)] if big else inputs.SHAPES_2B
    token_counts = (1, 4, 16, 32, 64) if big else (1, 4, 16, 64, 128, 256, 512)
    rows = decode_rows(torch, b, peaks, shapes, token_counts, big=big, cold=True)
    b.sbn_check_status()
    print(json.dumps({"metric": "small-T sparse vs dense ternary BitLinear, HBM GB/s (cold L2)", "unit": "GB/s",
                      "workload": args.workload, "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
                      "rows": rows, "gpu_launches": b.sbn_launch_count()}))


def run_pattern68(args):
    """The 6:8 pattern (the paper's deployed pattern) next to 2:4 and dense on the same matrices:
    per layer the isolated kernels with a cold L2 (pack, activation quantiser, GEMM), and the
    whole step (pack + quantise + GEMM for all layers) back to back.  Work is counted as the dense
    2 T N K whatever the pattern, so TOPS compare directly.  6:8 runs as 2:4 over 3K/2 expanded
    columns: 3/4 of the dense MMA work."""
    import torch
    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build
    sbn_build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    stream = torch.cuda.current_stream()
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    time_cold = _cold_timer(torch, stream, flush)
    cases = [(n, K, N, 4096) for n, K, N in inputs.SHAPES_2B] + [("down_7b", 11008, 4096, 8192)]
    if args.only_step:                      # profiler runs: the one 7B-class layer only
        cases = cases[-1:]
    rows, layers = [], []
    for i, (name, K, N, T) in enumerate(cases):
        W = torch.from_numpy(inputs.latent_weights(N, K, seed=1 + i)).cuda()
        x = torch.from_numpy(inputs.activations_bf16(T, K, seed=11 + i).view(np.int16)).cuda().view(torch.bfloat16)
        p24 = b.alloc_packed(N, K, with_dense=True)
        p68 = b.alloc_packed(N, K, n_keep=6, m_group=8)
        Kp = b.sbn_expanded_k(K, 6, 8)
        xq, xq68 = b.alloc_xq(T, K), b.alloc_xq(T, Kp)
        a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
        y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        ws24 = b.alloc_gemm_ws(b.OP_SPARSE_BITLINEAR, T, N, K)
        ws68 = b.alloc_gemm_ws(b.OP_SPARSE_BITLINEAR, T, N, Kp)
        wsd = b.alloc_gemm_ws(b.OP_BITLINEAR, T, N, K)
        f = {
            "pack24": lambda W=W, p=p24: b.sbn_quantize_mask_pack(W, p["vals"], p["meta"], p["w_scale"], p["ws"]),
            "pack68": lambda W=W, p=p68: b.sbn_quantize_mask_pack(W, p["vals"], p["meta"], p["w_scale"], p["ws"], n_keep=6, m_group=8),
            "act": lambda x=x, xq=xq, a=a_scale: b.sbn_quant_act(x, xq, a),
            "act68": lambda x=x, xq=xq68, a=a_scale: b.sbn_quant_act_expand68(x, xq, a),
            "gemm24": lambda xq=xq, a=a_scale, p=p24, y=y, ws=ws24: b.sbn_sparse_bitlinear(xq, a, p["vals"], p["meta"], p["w_scale"], y, ws=ws),
            "gemm68": lambda xq=xq68, a=a_scale, p=p68, y=y, ws=ws68: b.sbn_sparse_bitlinear(xq, a, p["vals"], p["meta"], p["w_scale"], y, ws=ws),
            "dense": lambda xq=xq, a=a_scale, p=p24, y=y, ws=wsd: b.sbn_bitlinear(xq, a, p["dense_q"], p["w_scale"], y, ws=ws),
        }
        b.sbn_quantize_mask_pack(W, p24["vals"], p24["meta"], p24["w_scale"], p24["ws"], dense_q=p24["dense_q"])
        for fn in f.values():
            for _ in range(3):
                fn()
        us = {k: time_cold(fn, 12) for k, fn in f.items()}
        ops = 2.0 * T * N * K
        rows.append({"layer": name, "T": T, "K": K, "N": N, **{k + "_us": round(v, 2) for k, v in us.items()},
                     "dense_tops": round(ops / us["dense"] / 1e6, 1), "sparse24_tops": round(ops / us["gemm24"] / 1e6, 1),
                     "sparse68_tops": round(ops / us["gemm68"] / 1e6, 1),
                     "speedup24_vs_dense": round(us["dense"] / us["gemm24"], 3),
                     "speedup68_vs_dense": round(us["dense"] / us["gemm68"], 3),
                     "pack68_gbs": round(N * K * (4 + 0.9375) / us["pack68"] / 1e3, 1),       # W once + 0.75 B vals + 0.1875 B meta
                     "act68_gbs": round((T * K * 3.5 + T * 4) / us["act68"] / 1e3, 1)})       # 2 B read + 1.5 B written
        if T == 4096:
            layers.append((f, ops))
    if not layers:
        b.sbn_check_status()
        print(json.dumps({"metric": "6:8 sparse ternary BitLinear next to 2:4 and dense (dense-equivalent TOPS)", "unit": "TOPS",
                          "workload": "p68", "rows": rows, "gpu_launches": b.sbn_launch_count()}))
        return

    # whole steps over the four 2B-shaped layers, back to back
    def step(kind):
        for f, _ in layers:
            if kind == "68":
                f["pack68"](); f["act68"](); f["gemm68"]()
            elif kind == "24":
                f["pack24"](); f["act"](); f["gemm24"]()
            else:
                f["act"](); f["dense"]()
    steps = {}
    for kind in ("68", "24", "dense_forward_only"):
        for _ in range(3):
            step(kind)
        torch.cuda.synchronize()
        torch.cuda._sleep(int(2e7))
        a = torch.cuda.Event(enable_timing=True)
        c = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.steps):
            step(kind)
        c.record(stream)
        torch.cuda.synchronize()
        steps[kind] = a.elapsed_time(c) / args.steps
    b.sbn_check_status()
    total_ops = sum(o for _, o in layers)
    print(json.dumps({"metric": "6:8 sparse ternary BitLinear next to 2:4 and dense (dense-equivalent TOPS)", "unit": "TOPS",
                      "workload": "p68", "rows": rows,
                      "step_ms": {k: round(v, 4) for k, v in steps.items()},
                      "step_tops": {k: round(total_ops / v / 1e9, 1) for k, v in steps.items()},
                      "note": "steps 68 / 24: one pack launch per layer (the headline step batches the 2:4 packs into one launch); "
                              "dense_forward_only: activation quantiser + dense GEMM, no packing",
                      "gpu_launches": b.sbn_launch_count()}))


def dyn_oracle_leg(torch, b, mats, host_W, host_x, acts, cur_meta, T):
    """The dynamic-mask step against the CPU oracle on the seven matrices of layer 0 (host-seeded): after
    the first timed step the scale, every packed byte (through the library's own un-tiling call) and the
    flip count of each matrix, and 2048 sampled outputs of each of its BitLinears.  Raises on a mismatch."""
    import oracle
    worst_ulp, checked = 0, 0
    for m_i in range(len(inputs.LAYER_2B)):
        name, K, N, W, p = mats[m_i]
        r_prev = oracle.quantize_mask_pack(host_W[("prev", m_i)])
        r = oracle.quantize_mask_pack(host_W[m_i])
        if r["near_tie"] or r_prev["near_tie"]:
            continue
        vals = torch.empty((N, K // 2), dtype=torch.int8, device="cuda")
        meta = torch.empty((N, K // 8), dtype=torch.uint8, device="cuda")
        b.sbn_unpack_canonical(p["vals"], cur_meta(p), N, K, vals, meta)
        b.sbn_check_status()
        if np.float32(p["w_scale"].cpu().numpy()[0]) != r["scale"]:
            raise RuntimeError(f"dyn oracle leg: scale of {name} differs from the oracle")
        if not (np.array_equal(vals.cpu().numpy(), r["vals"]) and np.array_equal(meta.cpu().numpy(), r["meta"])):
            raise RuntimeError(f"dyn oracle leg: packed weights of {name} differ from the oracle")
        want_flips = oracle.flip_count(r_prev["mask"], r["mask"])
        if int(p["flips"].item()) != want_flips:
            raise RuntimeError(f"dyn oracle leg: flip count of {name}: {int(p['flips'].item())} != oracle {want_flips}")
        xq_ref, s_ref = oracle.quant_act(host_x[K])
        xq, a_scale = acts[K]
        y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        b.sbn_sparse_bitlinear(xq, a_scale, p["vals"], cur_meta(p), p["w_scale"], y)
        b.sbn_check_status()
        t_idx, n_idx = inputs.sample_positions(T, N, 2048, seed=900 + m_i)
        acc_ref = oracle.acc_packed_sampled(xq_ref, r["vals"], r["meta"], t_idx, n_idx)
        y_ref = oracle.dequant(acc_ref.reshape(-1, 1), r["scale"], s_ref[t_idx]).ravel()
        got = y.view(torch.int16).cpu().numpy().view(np.uint16)[t_idx, n_idx].astype(np.int32)
        ulp = int(np.abs(got - oracle.f32_to_bf16_bits(y_ref).astype(np.int32)).max())
        if ulp > 1:
            raise RuntimeError(f"dyn oracle leg: outputs of {name} off by {ulp} bf16 ulp")
        worst_ulp = max(worst_ulp, ulp)
        checked += 1
    return {"layer": 0, "matrices_checked": checked, "checked": "w_scale, vals, meta, flip count (all exact); 2048 sampled bf16 outputs per BitLinear",
            "max_output_ulp": worst_ulp}


def run_dynamic_step(args):
    """Dynamic-mask training step (the mask is recomputed every step): perturb all master weights
    (outside the timed region), then timed: quantise/mask/pack all 30 x 7 matrices with the flip
    count against the previous step's metadata, then all 210 sparse BitLinears at T = 2048."""
    import torch
    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build
    sbn_build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    T, n_layers = 2048, 30
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    mats = []
    # Oracle leg: the seven matrices of layer 0 are drawn (and perturbed) on the HOST with the seeded
    # generators of inputs.py, so the CPU oracle sees the very same weights; the other 29 layers are drawn
    # on the device (8 GB of host-generated weights would dominate the run).
    oracle_leg = args.masters == "fp32" and not args.no_cpu_baseline
    host_W = {}
    for layer in range(n_layers):
        for j, (name, K, N) in enumerate(inputs.LAYER_2B):
            if layer == 0 and oracle_leg:
                host_W[j] = inputs.latent_weights(N, K, seed=700 + j)
                W = torch.from_numpy(host_W[j]).cuda()
            else:
                W = torch.randn((N, K), generator=gen, device="cuda", dtype=torch.float32) * 0.02
            if args.masters == "bf16":
                W = W.to(torch.bfloat16)
            p = b.alloc_packed(N, K)
            p["prev"] = torch.empty_like(p["meta"])
            p["flips"] = torch.zeros(1, dtype=torch.int64, device="cuda")
            mats.append((name, K, N, W, p))
    # one activation set per distinct K (shared by the layers; attention/norms are not on this path)
    acts, host_x = {}, {}
    for K in sorted({K for _, K, _ in inputs.LAYER_2B}):
        host_x[K] = inputs.activations_bf16(T, K, seed=750 + K)
        x = torch.from_numpy(host_x[K].view(np.int16)).cuda().view(torch.bfloat16)
        xq = b.alloc_xq(T, K)
        a_scale = torch.empty(T, dtype=torch.float32, device="cuda")
        b.sbn_quant_act(x, xq, a_scale)
        acts[K] = (xq, a_scale)
    ys = {N: torch.empty((T, N), dtype=torch.bfloat16, device="cuda") for N in sorted({N for _, _, N in inputs.LAYER_2B})}
    params = sum(K * N for _, K, N, _, _ in mats)

    # one batched launch per step; two job arrays because prev/current metadata swap every step
    job_ws = torch.empty(b.sbn_batch_workspace_bytes(len(mats)), dtype=torch.uint8, device="cuda")
    plain_jobs = b.make_pack_jobs([dict(W=W, vals=p["vals"], meta=p["meta"], w_scale=p["w_scale"]) for _, _, _, W, p in mats])
    flip_jobs = [b.make_pack_jobs([dict(W=W, vals=p["vals"], meta=p["meta"] if par == 0 else p["prev"], w_scale=p["w_scale"],
                                        prev_meta=p["prev"] if par == 0 else p["meta"], flip_bits=p["flips"],
                                        gamma_hint=p["w_scale"])              # the previous step's scale
                                   for _, _, _, W, p in mats]) for par in (0, 1)]
    state = {"par": 1}            # after the plain pack the current metadata is in p["meta"]

    def repack(with_flips):
        if not with_flips:
            b.sbn_quantize_mask_pack_batched(plain_jobs, job_ws)
            return
        b.sbn_quantize_mask_pack_batched(flip_jobs[state["par"]], job_ws)
        state["par"] ^= 1

    def cur_meta(p):
        return p["meta"] if state["par"] == 1 else p["prev"]

    def forward():
        for _, K, N, W, p in mats:
            xq, a_scale = acts[K]
            b.sbn_sparse_bitlinear(xq, a_scale, p["vals"], cur_meta(p), p["w_scale"], ys[N])

    repack(False)
    forward()
    b.sbn_check_status()
    rep_ms, fwd_ms, rates = [], [], []
    steps = max(1, min(args.steps, 5))
    oracle_report = None
    for s_i in range(steps + 1):
        for m_i, (_, K, N, W, p) in enumerate(mats):              # the optimiser step stand-in
            if m_i in host_W and s_i <= 1:
                # layer 0 up to the checked step: the perturbation is drawn on the host, like the weights
                host_prev = host_W[m_i]
                host_W[m_i] = inputs.perturb_weights(host_prev, seed=800 + 10 * s_i + m_i, sigma=1e-4)
                W.copy_(torch.from_numpy(host_W[m_i]))
                if s_i == 1:
                    host_W[("prev", m_i)] = host_prev
            else:
                W.add_(torch.randn(W.shape, generator=gen, device="cuda", dtype=torch.float32).to(W.dtype), alpha=1e-4)
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        torch.cuda._sleep(int(4e7))
        e[0].record(stream)
        repack(True)
        e[1].record(stream)
        forward()
        e[2].record(stream)
        torch.cuda.synchronize()
        if s_i == 0:
            continue                                              # warm-up step
        rep_ms.append(e[0].elapsed_time(e[1]))
        fwd_ms.append(e[1].elapsed_time(e[2]))
        flips = sum(int(p["flips"].item()) for *_, p in mats)
        rates.append(flips / params)
        if s_i == 1 and oracle_leg:
            oracle_report = dyn_oracle_leg(torch, b, mats, host_W, host_x, acts, cur_meta, T)
    b.sbn_check_status()
    rep, fwd = statistics.median(rep_ms), statistics.median(fwd_ms)
    fwd_ops = sum(2.0 * T * N * K for _, K, N, _, _ in mats)
    print(json.dumps({
        "metric": "dynamic-mask training step latency (re-pack 210 matrices + 210 sparse BitLinears at T=2048)",
        "unit": "ms", "workload": "dyn", "value": rep + fwd, "higher_is_better": False,
        "repack_ms": round(rep, 3), "forward_ms": round(fwd, 3), "params": params,
        "masters": args.masters,
        "repack_gbs_algorithmic": round(params * ((2 if args.masters == "bf16" else 4) + 0.75) / (rep * 1e-3) / 1e9, 1),   # W read + 0.625 written + 0.125 prev meta
        "repack_frac_of_hbm": round(params * ((2 if args.masters == "bf16" else 4) + 0.75) / (rep * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
        "forward_tops": round(fwd_ops / (fwd * 1e-3) / 1e12, 1),
        "forward_pct_sparse_int8_datasheet": round(100 * fwd_ops / (fwd * 1e-3) / 1e12 / DATASHEET_INT8_SPARSE_TOPS, 1),
        "flip_rate": statistics.mean(rates), "steps": steps,
        "data": "synthetic: layer 0 and all activations seeded on the host (inputs.py), layers 1-29 from torch's CUDA generator (seed 1234)",
        "oracle_leg": oracle_report,
        "gpu_launches": b.sbn_launch_count()}))


def run_backward(args):
    """The layer's backward (dual straight-through estimator) on the four 2B-shaped layers at T = 4096 (see
    backward_rows); --only-step: the qkv shape alone, a few calls (the small case for profiler runs)."""
    import torch
    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build
    sbn_build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    shapes = inputs.SHAPES_2B[:1] if args.only_step else inputs.SHAPES_2B
    layers = [Layer(n, K, N, T_TOKENS, seed=1 + i, torch=torch, b=b) for i, (n, K, N) in enumerate(shapes)]
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    rows = backward_rows(torch, b, peaks, layers, _cold_timer(torch, stream, flush), 3 if args.only_step else 12)
    print(json.dumps({"metric": "dual-STE backward of one Sparse-BitLinear layer: dX = dY w_masked, dW = dY^T x_q (bf16, fp32 accumulation)",
                      "unit": "us", "workload": "bwd", "tokens": T_TOKENS, "rows": rows,
                      "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TFLOP/s", "gpu_launches": b.sbn_launch_count()}))


def run_mma_probe(args):
    """What the K-loop of the large-T GEMM kernel costs, piece by piece (timing only: with a probe flag set
    the kernel's results are wrong).  One tile per CTA pair (74 feature tiles x one token tile), so nothing
    but the K-loop grows with K (two feature tiles x 37 token tiles, so operands are shared between pairs
    through the L2 as in a real layer); the time per 128-column block is the slope between K = 2560 and K = 11008.
    Modes: all loads | operands resident after the first fill | no loads | no loads and no metadata copies |
    no loads, every MMA issued twice / four times (the extra MMAs re-read operands the tensor core has just
    used: their marginal cost is the pipe's own pace)."""
    import torch
    from paper_2603_05168_b200 import binding as b
    from paper_2603_05168_b200 import build as sbn_build
    sbn_build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    stream = torch.cuda.current_stream()
    K1, K2 = 2560, 11008
    modes = [("all loads", 0), ("resident", 1), ("no loads", 6), ("no loads, no metadata copies", 14),
             ("no loads, MMAs x2", 14 + 16), ("no loads, MMAs x4", 14 + 32)]
    rows = []

    def timed(fn, reps=6):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            c.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(c) * 1e3)
        return statistics.median(ts)

    for sparse in (True, False):
        for mt in (1, 2):
            N = 2 * 256 * mt
            bufs = {}
            for K in (K1, K2):
                w = (torch.zeros((N, K // 2), dtype=torch.int8, device="cuda"), torch.full((N, K // 8), 0x44, dtype=torch.uint8, device="cuda")) \
                    if sparse else (torch.zeros((N, K), dtype=torch.int8, device="cuda"), None)
                bufs[K] = w
            w_scale = torch.ones(1, dtype=torch.float32, device="cuda")
            for bn in (64, 128, 240):
                T = 37 * bn
                b.sbn_set_gemm_tuning(-bn, 1 if mt == 1 else 0)
                y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
                a_scale = torch.ones(T, dtype=torch.float32, device="cuda")
                xq = {K: torch.zeros(b.sbn_xq_bytes(T, K), dtype=torch.int8, device="cuda") for K in (K1, K2)}
                for name, flags in modes:
                    if not sparse and (flags & 8) and not (flags & 48):
                        continue                                   # the dense kernel has no metadata copies
                    b.sbn_set_gemm_probe(flags)
                    t = {}
                    for K in (K1, K2):
                        if sparse:
                            fn = lambda K=K: b.sbn_sparse_bitlinear(xq[K], a_scale, bufs[K][0], bufs[K][1], w_scale, y)
                        else:
                            fn = lambda K=K: b.sbn_bitlinear(xq[K], a_scale, bufs[K][0], w_scale, y)
                        t[K] = timed(fn)
                    b.sbn_set_gemm_probe(0)
                    us_kb = (t[K2] - t[K1]) / ((K2 - K1) / 128)
                    reps = 4 if flags & 32 else (2 if flags & 16 else 1)
                    mmas_per_kb = (2 if sparse else 4) * mt * reps
                    rows.append({"kernel": ("sparse" if sparse else "dense") + f", {mt} M-tile(s) per CTA", "tokens_per_tile": bn, "mode": name,
                                 "us_per_128_columns": round(us_kb, 4), "mmas_per_128_columns": mmas_per_kb,
                                 "clocks_per_mma_at_1965mhz": round(us_kb * 1965.0 / mmas_per_kb, 1),
                                 "us_K2560": round(t[K1], 2), "us_K11008": round(t[K2], 2)})
                b.sbn_set_gemm_tuning(0, 0)
            del bufs
            torch.cuda.empty_cache()
    b.sbn_check_status()
    print(json.dumps({"metric": "K-loop cost of the CTA-pair GEMM kernel per 128 columns, by parts (timing experiments)", "unit": "us",
                      "workload": "mmaprobe", "note": "one tile per CTA pair (2 feature tiles x 37 token tiles); slope between K = 2560 and K = 11008; the math of one MMA "
                      "(M = 256 per pair, N tokens, K = 64 sparse / 32 dense) takes 128 clocks at N = 256 at the datasheet rate",
                      "rows": rows, "gpu_launches": b.sbn_launch_count()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="headline line only: skip the 7B-class isolated GEMMs, the sustained run and the few-token rows")
    ap.add_argument("--workload", default="2b", choices=sorted(WORKLOADS) + ["decode", "decode7b", "dyn", "p68", "mmaprobe", "bwd"],
                    help="2b = the headline workload; 7b / down7b = 7B-class shapes (down7b: one layer, for profiling); "
                         "decode = small-T sweep (T in 1..512), sparse vs dense, cold L2 and streamed; "
                         "decode7b = the same on 7B-class matrices at T <= 64, with the 2-bit packed weights as a third arm; "
                         "dyn = dynamic-mask training step: re-pack 30 x 7 matrices + forward at T=2048; "
                         "p68 = the 6:8 pattern next to 2:4 and dense on the same matrices; "
                         "mmaprobe = timing experiments on the large-T kernel's K-loop (loads, metadata copies, MMA issue); "
                         "bwd = the layer's backward (dual straight-through estimator) on the 2B shapes")
    ap.add_argument("--masters", default="fp32", choices=["fp32", "bf16"],
                    help="precision of the master weights the pack kernel reads (default fp32, the configuration of the metric)")
    ap.add_argument("--only-step", action="store_true", help="time the step only (used for profiler runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload in ("decode", "decode7b"):
        run_decode_sweep(args)
    elif args.workload == "dyn":
        run_dynamic_step(args)
    elif args.workload == "p68":
        run_pattern68(args)
    elif args.workload == "mmaprobe":
        run_mma_probe(args)
    elif args.workload == "bwd":
        run_backward(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
