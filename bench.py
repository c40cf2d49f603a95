#!/usr/bin/env python
"""Benchmark of the fused-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode fwd|fwd_bwd]
    python bench.py --impl reference ...        # times the fp64 CPU oracle on the same workload

One "step" is one pass of the path over one batch of synthetic inputs: for the default workload
(the forward-only microbenchmark shape B=4, H=16, S=8192, D=128, non-causal, on which the
throughput target is stated) that is one ``vt_attn_fwd`` call; with ``--mode fwd_bwd`` it is
``vt_attn_fwd`` followed by ``vt_attn_bwd``.  Prints ONE JSON line on rank 0.

Timing: CUDA events on the launching stream around K back-to-back steps after W warm-ups, a barrier
and a device synchronise on both sides, max over ranks.  The inputs of every workload timed here
are larger than L2 or, for the small ones, L2 is flushed between steps (stated in ``config``).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_16238_b200.dist import (barrier, env_rank_world, init_process_group,  # noqa: E402
                                        max_over_ranks)
from paper_2601_16238_b200.inputs import (CONFIGS, VARLEN_CONFIGS, make_inputs,  # noqa: E402
                                          make_varlen_inputs)

DATASHEET_BF16_TFLOPS = 2250.0
# The paper's own latencies (its best kernel, H100 PCIe) for the one attention workload it reports: the rows
# "Attention (fwd)" and "Attention (bwd)" of its kernel microbenchmark table, shape (32, 10, 10, 2048, 128) bf16 causal.
PAPER_MS = {"paper_shape": {"fwd": 1.46, "fwd_bwd": 1.46 + 6.97}}


def paper_ratio(workload, mode, ms):
    """value / the paper's number for the same metric and workload (same flop count, so the ratio of the times); None
    where the paper has no number.  Another machine's figure: context, not a target."""
    ref = PAPER_MS.get(workload, {}).get(mode)
    return ref / ms if ref else None

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 1024 * 1024

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant
# kernel, from the ncu captures summarised under profiles/; None where no capture exists.
NCU_TRAFFIC_BYTES = {
    # profiles/attn_fwd_pair_kernel_sdpa_s8192_nc.md: 402.7 MB read + 115.0 MB written, one launch at full size
    "sdpa_s8192_nc": 517.7e6,
    # profiles/attn_fwd_pair_kernel_sdpa_s4096_nc.md: 201.4 MB read + 50.0 MB written per launch
    "sdpa_s4096_nc": 251.4e6,
    # profiles/attn_fwd_kernel_paper_shape.md: 504.0 MB read + 156.3 MB written
    "paper_shape": 660.3e6,
    # profiles/launch_lists.md, decoding: split-KV kernel 537.0 + 1.3 MB, merge kernel 0.6 MB per step
    "decode_32k": 538.9e6,
    # profiles/bwd_kernels_gqa_long.md, one launch of each kernel at full size: forward 312.3 MB; backward
    # (Delta 273.9 + dK/dV 397.4 + dQ 454.0 MB)
    "gqa_long": 312.3e6,
    "gqa_long_bwd": 1125.3e6,
    # profiles/attn_fwd_kernel_d64_s4096_nc.md: 101.1 MB read + 17.3 MB written (part of O still in L2 at the end)
    "d64_s4096_nc": 118.4e6,
    # profiles/fwd_bwd_kernels_d256_s4096_nc.md: forward 201.5 MB read + 48.0 MB written
    "d256_s4096_nc": 249.5e6,
}
NCU_TRAFFIC_NOTE = {}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80, "sw_power_cap": 0x4}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def device_tensors(cfg, torch, with_do, f16=False):
    """Seeded inputs on the device: the shared bf16 bit patterns, or (f16) the same seeds' N(0,1) values rounded to fp16."""
    if f16:
        from paper_2601_16238_b200.inputs import normal_f16
        base = 1000 * cfg.index
        shapes = [(cfg.B, cfg.Hq, cfg.Sq, cfg.D), (cfg.B, cfg.Hkv, cfg.Sk, cfg.D), (cfg.B, cfg.Hkv, cfg.Sk, cfg.D)]
        if with_do:
            shapes.append((cfg.B, cfg.Hq, cfg.Sq, cfg.D))
        return [torch.from_numpy(normal_f16(sh, base + 1 + i).view(np.int16)).view(torch.float16).cuda() for i, sh in enumerate(shapes)]
    bits = make_inputs(cfg, with_do=with_do)
    return [torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda() for x in bits]


def algorithmic_bytes(cfg, mode):
    """Bytes a perfect kernel moves: every input read once, every output written once."""
    qb = cfg.B * cfg.Hq * cfg.Sq * cfg.D * 2
    kvb = cfg.B * cfg.Hkv * cfg.Sk * cfg.D * 2
    lse = cfg.B * cfg.Hq * cfg.Sq * 4
    fwd = qb + 2 * kvb + qb + lse
    if mode == "fwd":
        return fwd
    return fwd + (3 * qb + 2 * kvb + lse) + (qb + 2 * kvb)     # + bwd reads q,o,do,k,v,lse + writes dq,dk,dv


def time_steps(torch, step, steps, warmup, flush=None):
    for _ in range(warmup):
        if flush is not None:
            flush()
        step()
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        total = e0.elapsed_time(e1)
    else:
        total = 0.0
        for _ in range(steps):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            step()
            e1.record(stream)
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
    barrier()
    return total / steps


def run_varlen(args):
    """Packed (variable-length) workloads: same contract, the step is vt_attn_fwd_varlen (+ vt_attn_bwd_varlen)."""
    import torch
    import paper_2601_16238_b200 as vt

    rank, local_rank, world = env_rank_world()
    torch.cuda.set_device(local_rank)
    init_process_group("nccl")
    vt.load_library()
    peaks, peak_kind = load_peaks()
    cfg = VARLEN_CONFIGS[args.workload]
    mode = args.mode or "fwd"
    with_bwd = mode == "fwd_bwd"
    bits = make_varlen_inputs(cfg, with_do=True)
    to_dev = lambda x: torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda()      # noqa: E731
    q, k, v, d_o = (to_dev(x) for x in bits[:4])
    cu = torch.from_numpy(bits[4]).cuda()
    lens = cfg.lengths()
    o = torch.empty_like(q)
    lse = torch.empty((cfg.Hq, cfg.total), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(max(256, vt.vt_attn_bwd_varlen_workspace_bytes(cfg.Hq, cfg.total)), dtype=torch.uint8, device="cuda")

    def step():
        vt.vt_attn_fwd_varlen(q, k, v, cu, cu, max(lens), max(lens), cfg.causal, cfg.scale, o, lse)
        if with_bwd:
            vt.vt_attn_bwd_varlen(q, k, v, o, d_o, lse, cu, cu, max(lens), max(lens), cfg.causal, cfg.scale, dq, dk, dv, ws)

    qb, kvb = q.numel() * 2, k.numel() * 2
    touched = 2 * qb + 2 * kvb + lse.numel() * 4 + ((3 * qb + 2 * kvb + lse.numel() * 4) + (qb + 2 * kvb) if with_bwd else 0)
    flush, l2_note = None, f"inputs+outputs {touched / 1e6:.0f} MB exceed the 126 MB L2"
    if touched <= 2 * L2_BYTES:
        # flushed by READING a buffer twice the size of L2: a write flush would leave dirty lines whose write-back lands
        # inside the timed kernels
        scratch = torch.zeros(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
        flush = lambda: scratch.max()      # noqa: E731
        l2_note = "L2 flushed (252 MB read) before every timed step"
    with ClockSampler(local_rank) as clocks:
        ms = time_steps(torch, step, args.steps, args.warmup, flush)
    rc, detail = vt.vt_attn_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} (detail {detail:#x}) after the timed region")
    ms = max_over_ranks(ms, device="cuda")
    flops = cfg.fwd_flops() * (3.5 if with_bwd else 1.0)
    tflops = flops / (ms * 1e-3) / 1e12

    # end to end: pinned host -> device copies of the step's inputs, kernels, device -> host copy of the results
    host_in = [t.cpu().pin_memory() for t in ((q, k, v, d_o) if with_bwd else (q, k, v))]
    dev_in = [q, k, v, d_o][:len(host_in)]
    outs = [o, lse] + ([dq, dk, dv] if with_bwd else [])
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in outs]

    def e2e_step():
        for h, d in zip(host_in, dev_in):
            d.copy_(h, non_blocking=True)
        step()
        for h, d in zip(host_out, outs):
            h.copy_(d, non_blocking=True)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms = max_over_ranks(time_steps(torch, e2e_step, e2e_steps, 3, None), device="cuda")
    if rank != 0:
        return
    peak = float(peaks["bf16_tflops"])
    info = vt.vt_attn_get_info()
    line = {
        "metric": f"fused attention {'fwd+bwd' if with_bwd else 'fwd'} TFLOP/s (bf16)", "value": tflops * world, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "layout": "packed [total, H, D] + cu_seqlens", "total_tokens": cfg.total,
                   "n_seqs": len(lens), "min_len": min(lens), "max_len": max(lens), "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "causal": cfg.causal, "mode": mode, "l2": l2_note,
                   "flops_convention": "sum over sequences of 4*Hq*S_i^2*D (x0.5 causal), bwd = 2.5x fwd",
                   "parallelism": f"dp{world} (batch shards, no collective)"},
        "pct_of_measured_bf16_peak": 100.0 * tflops / peak, "pct_of_datasheet_bf16_peak": 100.0 * tflops / DATASHEET_BF16_TFLOPS,
        "clocks": clocks.summary(),
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12 * world, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_in)),
                "d2h_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_out)), "steps": e2e_steps,
                "api": "torch pinned copies + vt_attn_fwd_varlen" + (" + vt_attn_bwd_varlen" if with_bwd else "")},
        "gpu_launches": (info[6] + (info[7] if with_bwd else 0)) * args.steps,
        "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel (packed)" if not with_bwd else "packed fwd + bwd kernels",
                     "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
                     "peak_kind": f"{peak_kind} cuBLAS bf16 burst", "traffic": None, "algorithmic_bytes": int(touched),
                     "hbm_gbs_at_algorithmic_bytes": touched / (ms * 1e-3) / 1e9},
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import attn_oracle as orc
        n_seq = max(1, min(len(lens), orc.num_threads()))         # a few whole documents
        end = int(bits[4][n_seq])
        t0 = time.perf_counter()
        orc.attn_fwd_varlen(bits[0][:end], bits[1][:end], bits[2][:end], bits[4][:n_seq + 1], bits[4][:n_seq + 1], cfg.causal, cfg.scale)
        if with_bwd:
            orc.attn_bwd_varlen(bits[0][:end], bits[1][:end], bits[2][:end], bits[3][:end], bits[4][:n_seq + 1], bits[4][:n_seq + 1],
                                cfg.causal, cfg.scale)
        sec = time.perf_counter() - t0
        sub = sum(4.0 * cfg.Hq * n * n * cfg.D for n in lens[:n_seq]) * (0.5 if cfg.causal else 1.0) * (3.5 if with_bwd else 1.0)
        line["cpu_baseline"] = {"value": sub / sec / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(), "kind": "oracle",
                                "seconds": sec, "sample": f"first {n_seq} documents ({end} tokens) of {cfg.name}, one after another"}
    print(json.dumps(line), flush=True)


# Ragged decoding: one new token per sequence against caches of different lengths (seeded, uniform in [1024, 32768]),
# 32 query heads on 8 KV heads, D = 128, through the packed split-KV entry point.  HBM-bound: K and V are read once.
DECODE_RAGGED = {"n_seqs": 16, "Hq": 32, "Hkv": 8, "D": 128, "min_len": 1024, "max_len": 32768, "seed": 77}


def run_decode_ragged(args):
    import torch
    import paper_2601_16238_b200 as vt
    from paper_2601_16238_b200.inputs import normal_bf16

    rank, local_rank, world = env_rank_world()
    torch.cuda.set_device(local_rank)
    init_process_group("nccl")
    vt.load_library()
    peaks, peak_kind = load_peaks()
    c = DECODE_RAGGED
    gen = np.random.Generator(np.random.Philox(key=c["seed"]))
    lens_k = [int(x) for x in gen.integers(c["min_len"], c["max_len"] + 1, c["n_seqs"])]
    n, Hq, Hkv, D = c["n_seqs"], c["Hq"], c["Hkv"], c["D"]
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    bits = [normal_bf16(s, 7100 + i) for i, s in enumerate(((n, Hq, D), (sum(lens_k), Hkv, D), (sum(lens_k), Hkv, D)))]
    q, k, v = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda() for x in bits)
    cu_q_h = np.arange(n + 1, dtype=np.int32)
    cu_k_h = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    cu_q, cu_k = torch.from_numpy(cu_q_h).cuda(), torch.from_numpy(cu_k_h).cuda()
    o = torch.empty_like(q)
    lse = torch.empty((Hq, n), dtype=torch.float32, device="cuda")
    need = vt.load_library().vt_attn_fwd_splitkv_varlen_workspace_bytes(n, Hq, Hkv, n, 1, max(lens_k), D, 0)
    ws = torch.empty(max(256, need), dtype=torch.uint8, device="cuda")
    step = lambda: vt.vt_attn_fwd_splitkv_varlen(q, k, v, cu_q, cu_k, 1, max(lens_k), 2, scale, 0, o, lse, ws)      # noqa: E731
    touched = 2 * k.numel() * 2 + 2 * q.numel() * 2 + lse.numel() * 4
    with ClockSampler(local_rank) as clocks:
        ms = max_over_ranks(time_steps(torch, step, args.steps, args.warmup, None), device="cuda")
    rc, detail = vt.vt_attn_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} (detail {detail:#x}) after the timed region")
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty_like(hq).pin_memory()

    def e2e_step():
        for h, d in ((hq, q), (hk, k), (hv, v)):
            d.copy_(h, non_blocking=True)
        step()
        ho.copy_(o, non_blocking=True)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms = max_over_ranks(time_steps(torch, e2e_step, e2e_steps, 3, None), device="cuda")
    if rank != 0:
        return
    flops = 4.0 * Hq * D * float(sum(lens_k))
    tflops = flops / (ms * 1e-3) / 1e12
    gbs = touched / (ms * 1e-3) / 1e9
    n_chunks, shared = vt.vt_attn_fwd_splitkv_varlen_plan(n, Hq, Hkv, sum(lens_k), 1, max(lens_k), D, 0)
    line = {
        "metric": "fused attention fwd TFLOP/s (bf16)", "value": tflops * world, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "decode_ragged", "layout": "packed [total, H, D] + cu_seqlens", "n_seqs": n, "Hq": Hq, "Hkv": Hkv, "D": D,
                   "cache_lengths": f"uniform in [{c['min_len']}, {c['max_len']}]: {min(lens_k)} .. {max(lens_k)}, {sum(lens_k)} keys in all",
                   "causal": 2, "mode": "fwd", "splitkv_chunks": n_chunks, "heads_share_a_tile": shared,
                   "l2": f"inputs {touched / 1e6:.0f} MB exceed the 126 MB L2", "parallelism": f"dp{world} (batch shards, no collective)"},
        "clocks": clocks.summary(),
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12 * world, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(sum(t.numel() * 2 for t in (hq, hk, hv))), "d2h_bytes_per_step": int(ho.numel() * 2),
                "steps": e2e_steps, "api": "torch pinned copies + vt_attn_fwd_splitkv_varlen"},
        "gpu_launches": 2 * args.steps,
        "roofline": {"bound": "hbm", "kernel": "attn_fwd_kernel (packed, split-KV, heads of a KV group in one tile) + fwd_merge_kernel",
                     "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]),
                     "peak_kind": f"{peak_kind} copy bandwidth", "traffic": None, "algorithmic_bytes": int(touched)},
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import attn_oracle as orc
        m = min(n, 4)                                      # the first few sequences, one after another
        t0 = time.perf_counter()
        orc.attn_fwd_varlen(bits[0][:m], bits[1][:cu_k_h[m]], bits[2][:cu_k_h[m]], cu_q_h[:m + 1], cu_k_h[:m + 1], 2, scale)
        sec = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 4.0 * Hq * D * float(sum(lens_k[:m])) / sec / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(),
                                "kind": "oracle", "seconds": sec, "sample": f"the first {m} sequences ({int(cu_k_h[m])} keys)"}
    print(json.dumps(line), flush=True)


def extra_fwd_bwd(torch, vt, peaks, local_rank, steps, warmup):
    """The forward + backward half of the metric, timed in the same run: the long-context GQA configuration
    (B = 1, 32 query heads on 8 KV heads, S = 16384, D = 128, causal), vt_attn_fwd followed by vt_attn_bwd."""
    cfg = CONFIGS["gqa_long"]
    q, k, v, d_o = device_tensors(cfg, torch, True)
    o = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D)
    ws = torch.empty(max(256, vt.vt_attn_bwd_workspace_bytes(*dims)), dtype=torch.uint8, device="cuda")

    def step():
        vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale, o, lse)
        vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)

    def bwd_only():
        vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)

    with ClockSampler(local_rank) as clocks:
        ms = max_over_ranks(time_steps(torch, step, steps, warmup, None), device="cuda")
    ms_bwd = max_over_ranks(time_steps(torch, bwd_only, steps, 1, None), device="cuda")
    rc, detail = vt.vt_attn_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} (detail {detail:#x}) after the forward + backward region")
    flops = cfg.fwd_flops() * 3.5
    tf = flops / (ms * 1e-3) / 1e12
    tf_bwd = cfg.bwd_flops() / (ms_bwd * 1e-3) / 1e12
    info = vt.vt_attn_get_info()
    touched = algorithmic_bytes(cfg, "fwd_bwd")
    return {"workload": cfg.name, "mode": "fwd_bwd", "ms_per_step": ms, "steps": steps, "warmup": warmup, "value": tf, "unit": "TFLOP/s",
            "frac_of_measured_burst_peak": tf / float(peaks["bf16_tflops"]),
            "frac_of_measured_sustained_peak": tf / float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])),
            "frac_of_datasheet_peak": tf / DATASHEET_BF16_TFLOPS,
            "backward_only": {"ms_per_step": ms_bwd, "value": tf_bwd, "frac_of_measured_burst_peak": tf_bwd / float(peaks["bf16_tflops"])},
            "gpu_launches": (info[6] + info[7]) * steps, "l2": f"inputs+outputs {touched / 1e6:.0f} MB exceed the 126 MB L2",
            "traffic": {"forward_kernel": NCU_TRAFFIC_BYTES.get("gqa_long"), "backward_kernels": NCU_TRAFFIC_BYTES.get("gqa_long_bwd"),
                        "source": "one ncu capture of each kernel at full size (profiles/bwd_kernels_gqa_long.md)"},
            "algorithmic_bytes": int(touched), "clocks": clocks.summary()}


def extra_sustained(torch, step, flops, peaks, local_rank, ms_hint, seconds=2.5):
    """The default workload back to back for at least `seconds` of device time (the power cap pulls the SM clock down
    after a few hundred milliseconds), with the median SM clock sampled meanwhile: time x MHz shows how the number
    depends on the clock without touching any setting."""
    n = max(20, int(seconds * 1e3 / max(ms_hint, 1e-3)) + 1)
    with ClockSampler(local_rank) as clocks:
        ms = max_over_ranks(time_steps(torch, step, n, 3, None), device="cuda")
    tf = flops / (ms * 1e-3) / 1e12
    c = clocks.summary()
    return {"steps": n, "ms_per_step": ms, "timed_seconds": n * ms * 1e-3, "value": tf, "unit": "TFLOP/s",
            "frac_of_measured_sustained_peak": tf / float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])),
            "frac_of_measured_burst_peak": tf / float(peaks["bf16_tflops"]),
            "ms_times_sm_mhz": (ms * c["sm_mhz"]) if c["sm_mhz"] else None, "clocks": c}


# ------------------------------------------------------------------------------------------------
# Context-parallel ring attention: one causal sequence sharded over the ranks in the zig-zag layout, forward + backward.
# The one workload with a real exchange step (K / V blocks and the running dK / dV travel around the ring with
# torch.distributed point-to-point operations: NCCL on GPUs); total work is fixed, so scaling is "strong".
# ------------------------------------------------------------------------------------------------
RING_WORKLOADS = {
    # name: B, Hq, Hkv, S (whole sequence), D; the sequence is generated in 16 seeded pieces so that every world size
    # (1, 2, 4, 8) sees the same data
    "ring_causal_64k": {"B": 1, "Hq": 32, "Hkv": 8, "S": 65536, "D": 128, "pieces": 16, "index": 31},
}


def ring_shard_bits(w, rank, world):
    """This rank's zig-zag shard of the workload's seeded inputs: four uint16 arrays [2, B, H, S_chunk, D] (q, k, v, dO)."""
    from paper_2601_16238_b200.inputs import normal_bf16
    from paper_2601_16238_b200.ring import zigzag_chunks
    if w["pieces"] % (2 * world) != 0:
        raise SystemExit(f"world size {world}: 2 * world must divide {w['pieces']}")
    per_chunk = w["pieces"] // (2 * world)
    rows = w["S"] // w["pieces"]
    out = []
    for t, heads in enumerate((w["Hq"], w["Hkv"], w["Hkv"], w["Hq"])):
        chunks = []
        for c in zigzag_chunks(rank, world):
            pieces = [normal_bf16((w["B"], heads, rows, w["D"]), 1000 * w["index"] + 100 * t + piece)
                      for piece in range(c * per_chunk, (c + 1) * per_chunk)]
            chunks.append(np.concatenate(pieces, axis=2))
        out.append(np.stack(chunks))
    return out


def ring_step(q2, k2, v2, do2, scale, group=None, comm_stream=None, **standins):
    """One step of the ring workload on this rank: causal forward + backward in the zig-zag layout."""
    from paper_2601_16238_b200.ring import ring_attention_zigzag_fwd_bwd
    return ring_attention_zigzag_fwd_bwd(q2, k2, v2, do2, scale, group, comm_stream, **standins)


def run_ring(args):
    import torch
    import paper_2601_16238_b200 as vt
    from paper_2601_16238_b200 import ring as ring_mod

    w = RING_WORKLOADS[args.workload]
    rank, local_rank, world = env_rank_world()
    torch.cuda.set_device(local_rank)
    init_process_group("nccl")
    vt.load_library()
    peaks, peak_kind = load_peaks()
    scale = float(np.float32(1.0) / np.sqrt(np.float32(w["D"])))
    bits = ring_shard_bits(w, rank, world)
    q2, k2, v2, do2 = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda() for x in bits)
    comm = torch.cuda.Stream() if world > 1 else None
    info = vt.vt_attn_get_info()
    launches = [0]

    def attend(q, k, v, mode, sc):                       # the library's kernels, counted
        launches[0] += info[6]
        return vt.vt_attn_fwd(q, k, v, mode, sc)

    def attend_bwd(q, k, v, o, d_o, lse, mode, sc):
        launches[0] += info[7]
        return vt.vt_attn_bwd(q, k, v, o, d_o, lse, mode, sc)

    class Merge(ring_mod._DeviceMerge):
        def add(self, o_part, lse_part):
            launches[0] += 1
            super().add(o_part, lse_part)

        def result(self):
            launches[0] += 1
            return super().result()

    class Sum(ring_mod._DeviceSum):
        def add(self, part):
            launches[0] += 1
            super().add(part)

        def result(self):
            launches[0] += 1
            return super().result()

    outs = [None]

    def step():
        outs[0] = ring_step(q2, k2, v2, do2, scale, None, comm, attend=attend, merge_factory=Merge, attend_bwd=attend_bwd, sum_factory=Sum)

    with ClockSampler(local_rank) as clocks:
        ms = max_over_ranks(time_steps(torch, step, args.steps, args.warmup, None), device="cuda")
    per_step_launches = launches[0] // (args.steps + args.warmup)
    rc, detail = vt.vt_attn_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} (detail {detail:#x}) after the timed region")
    flops = 4.0 * w["B"] * w["Hq"] * float(w["S"]) ** 2 * w["D"] * 0.5 * 3.5
    tflops = flops / (ms * 1e-3) / 1e12

    # end to end: this rank's shards start in pinned host memory, its results end there
    host_in = [t.cpu().pin_memory() for t in (q2, k2, v2, do2)]
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in outs[0]]

    def e2e_step():
        for h, d in zip(host_in, (q2, k2, v2, do2)):
            d.copy_(h, non_blocking=True)
        step()
        for h, d in zip(host_out, outs[0]):
            h.copy_(d, non_blocking=True)
    e2e_steps = max(3, min(args.steps, 5))
    e2e_ms = max_over_ranks(time_steps(torch, e2e_step, e2e_steps, 3, None), device="cuda")
    if rank != 0:
        return
    peak = float(peaks["bf16_tflops"])
    shard_bytes = sum(t.numel() * t.element_size() for t in (k2, v2))
    line = {
        "metric": "fused attention fwd+bwd TFLOP/s (bf16)", "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "B": w["B"], "Hq": w["Hq"], "Hkv": w["Hkv"], "S": w["S"], "D": w["D"], "causal": True,
                   "mode": "fwd_bwd", "layout": f"zig-zag: rank r holds chunks r and {2 * world - 1} - r of {2 * world}",
                   "exchange": "none (one rank)" if world == 1 else
                               f"torch.distributed point-to-point (NCCL) on its own stream: {shard_bytes / 1e6:.1f} MB of K/V per step forward, "
                               f"that plus {2 * shard_bytes / 1e6:.1f} MB of fp32 dK/dV sums per step backward",
                   "l2": "inputs exceed the 126 MB L2", "flops_convention": "4*B*Hq*S^2*D*0.5 forward, backward 2.5x",
                   "parallelism": f"cp{world} (sequence shards, ring exchange)"},
        "pct_of_measured_bf16_peak": 100.0 * tflops / (peak * world), "clocks": clocks.summary(),
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_in)) * world,
                "d2h_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_out)) * world, "steps": e2e_steps,
                "api": "pinned copies + ring_attention_zigzag_fwd_bwd"},
        "gpu_launches": per_step_launches * args.steps,
        "roofline": {"bound": "tensor", "kernel": "forward / backward attention kernels per block + merge and accumulate kernels",
                     "achieved": tflops / world, "peak": peak, "unit": "TFLOP/s", "frac": tflops / world / peak,
                     "peak_kind": f"{peak_kind} cuBLAS bf16 burst, per GPU", "traffic": None},
    }
    if world == 1 and not args.no_cpu_baseline and not args.lean:
        from paper_2601_16238_b200.inputs import AttnConfig
        cfg = AttnConfig(args.workload, w["index"], w["B"], w["Hq"], w["Hkv"], w["S"], w["S"], w["D"], True, True)
        line["cpu_baseline"] = cpu_baseline(cfg, True, budget_s=args.cpu_budget)
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import paper_2601_16238_b200 as vt

    if args.workload in VARLEN_CONFIGS:
        return run_varlen(args)
    if args.workload in RING_WORKLOADS:
        return run_ring(args)
    if args.workload == "decode_ragged":
        return run_decode_ragged(args)

    rank, local_rank, world = env_rank_world()
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    init_process_group("nccl")
    vt.load_library()                       # raises if the CUDA library is missing: no fallback
    peaks, peak_kind = load_peaks()

    cfg = CONFIGS[args.workload]
    mode = args.mode or "fwd"
    if mode == "fwd_bwd" and not cfg.backward:
        cfg = cfg.with_(backward=True)
    with_bwd = mode == "fwd_bwd"
    f16 = args.dtype == "f16"
    fwd_call, bwd_call = (vt.vt_attn_fwd_f16, vt.vt_attn_bwd_f16) if f16 else (vt.vt_attn_fwd, vt.vt_attn_bwd)
    tens = device_tensors(cfg, torch, with_bwd, f16)
    q, k, v = tens[:3]
    d_o = tens[3] if with_bwd else None
    o = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D)
    if with_bwd:
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        ws = torch.empty(max(256, vt.vt_attn_bwd_workspace_bytes(*dims)), dtype=torch.uint8, device="cuda")

    # low-occupancy forward shapes go through the split-KV entry point (the library's own plan says whether it would split)
    n_chunks, shared_tile = vt.vt_attn_fwd_splitkv_plan(*dims, 0)
    use_split = (not with_bwd) and (not f16) and args.splitkv != "off" and (args.splitkv == "on" or n_chunks > 1 or shared_tile)
    if use_split:
        split_ws = torch.empty(max(256, vt.load_library().vt_attn_fwd_splitkv_workspace_bytes(*dims, 0)), dtype=torch.uint8, device="cuda")

    def step():
        if use_split:
            vt.vt_attn_fwd_splitkv(q, k, v, cfg.causal, cfg.scale, 0, o, lse, split_ws)
            return
        fwd_call(q, k, v, cfg.causal, cfg.scale, o, lse)
        if with_bwd:
            bwd_call(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)

    touched = algorithmic_bytes(cfg, mode)
    flush = None
    l2_note = f"inputs+outputs {touched / 1e6:.0f} MB exceed the 126 MB L2"
    if touched <= 2 * L2_BYTES:
        # flushed by READING a buffer twice the size of L2: a write flush would leave dirty lines whose write-back lands
        # inside the timed kernels
        scratch = torch.zeros(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
        flush = lambda: scratch.max()      # noqa: E731
        l2_note = "L2 flushed (252 MB read) before every timed step"

    info = vt.vt_attn_get_info()
    launches_per_step = 2 if use_split else info[6] + (info[7] if with_bwd else 0)      # split: chunk kernel + merge
    timed_step = step
    if args.graph:
        # one step's kernels captured once into a CUDA graph and replayed: for steps of a few microseconds the host's
        # per-call work (argument checks, tensor-map lookup, launch) otherwise sets the pace, not the GPU
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        timed_step = graph.replay
    with ClockSampler(local_rank) as clocks:
        ms = time_steps(torch, timed_step, args.steps, args.warmup, flush)
    rc, detail = vt.vt_attn_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} (detail {detail:#x}) after the timed region")
    ms = max_over_ranks(ms, device="cuda")
    flops = cfg.fwd_flops() * (3.5 if with_bwd else 1.0)
    tflops_per_gpu = flops / (ms * 1e-3) / 1e12
    value = tflops_per_gpu * world

    # ---- the default line also carries the forward + backward half of the metric and a sustained figure
    extras = {}
    if args.workload == "sdpa_s8192_nc" and mode == "fwd" and not f16 and not args.lean:
        burst_clocks = clocks.summary()
        extras["sustained"] = extra_sustained(torch, timed_step, flops, peaks, local_rank, ms)
        extras["sustained"]["burst_ms_times_sm_mhz"] = (ms * burst_clocks["sm_mhz"]) if burst_clocks["sm_mhz"] else None
        torch.cuda.synchronize()
        time.sleep(1.0)                      # let the clock recover before the next burst-sized region
        extras["fwd_bwd"] = extra_fwd_bwd(torch, vt, peaks, local_rank, max(5, min(args.steps, 20)), 3)

    # ---- end to end through the host-buffer entry point: pinned host -> device -> kernels -> host
    e2e = None
    if (rank == 0 or world > 1) and not args.lean:
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        ho, hlse = torch.empty_like(hq).pin_memory(), torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        staging = torch.empty(vt.vt_attn_host_staging_bytes(*dims, with_bwd), dtype=torch.uint8, device="cuda")
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
        d2h = ho.numel() * 2 + hlse.numel() * 4
        if with_bwd:
            hdo = d_o.cpu().pin_memory()
            hdq, hdk, hdv = torch.empty_like(hq).pin_memory(), torch.empty_like(hk).pin_memory(), torch.empty_like(hv).pin_memory()
            h2d += hdo.numel() * 2
            d2h += (hdq.numel() + hdk.numel() + hdv.numel()) * 2

            if f16:
                def e2e_step():      # the host-buffer entry points are bf16-only: pinned copies around the device calls
                    q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True); d_o.copy_(hdo, non_blocking=True)
                    fwd_call(q, k, v, cfg.causal, cfg.scale, o, lse)
                    bwd_call(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)
                    ho.copy_(o, non_blocking=True); hlse.copy_(lse, non_blocking=True)
                    hdq.copy_(dq, non_blocking=True); hdk.copy_(dk, non_blocking=True); hdv.copy_(dv, non_blocking=True)
            else:
                def e2e_step():
                    vt.vt_attn_fwd_bwd_host(hq, hk, hv, hdo, ho, hlse, hdq, hdk, hdv, cfg.causal, cfg.scale, staging)
        elif f16:
            def e2e_step():
                q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True)
                fwd_call(q, k, v, cfg.causal, cfg.scale, o, lse)
                ho.copy_(o, non_blocking=True); hlse.copy_(lse, non_blocking=True)
        elif use_split:
            def e2e_step():      # pinned host -> device copies, the split-KV call, device -> pinned host copies
                q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True)
                vt.vt_attn_fwd_splitkv(q, k, v, cfg.causal, cfg.scale, 0, o, lse, split_ws)
                ho.copy_(o, non_blocking=True); hlse.copy_(lse, non_blocking=True)
        else:
            def e2e_step():
                vt.vt_attn_fwd_host(hq, hk, hv, ho, hlse, cfg.causal, cfg.scale, staging)
        e2e_steps = max(3, min(args.steps, 10))
        e2e_ms = time_steps(torch, e2e_step, e2e_steps, 3, None)
        e2e_ms = max_over_ranks(e2e_ms, device="cuda")
        e2e = {"value": flops / (e2e_ms * 1e-3) / 1e12 * world, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
               "api": ("pinned copies + vt_attn_fwd_f16" + (" + vt_attn_bwd_f16" if with_bwd else "")) if f16 else
                      ("vt_attn_fwd_bwd_host" if with_bwd else ("pinned copies + vt_attn_fwd_splitkv" if use_split else "vt_attn_fwd_host"))}

    if rank != 0:
        return
    peak = float(peaks["bf16_tflops"])
    fwd_kernel = ("attn_fwd_kernel", "attn_fwd_pair_kernel", "attn_fwd_duo_kernel")[vt.vt_attn_fwd_kernel_kind(*dims, cfg.causal)]
    roofline = {"bound": "tensor", "kernel": fwd_kernel if not with_bwd else f"{fwd_kernel} + bwd_delta / bwd_dkdv / bwd_dq kernels",
                "achieved": tflops_per_gpu, "peak": peak, "unit": "TFLOP/s", "frac": tflops_per_gpu / peak,
                "peak_kind": f"{peak_kind} cuBLAS bf16 burst", "traffic": NCU_TRAFFIC_BYTES.get(cfg.name),
                "algorithmic_bytes": int(touched), "hbm_gbs_at_algorithmic_bytes": touched / (ms * 1e-3) / 1e9,
                "frac_of_sustained_peak": tflops_per_gpu / float(peaks.get("bf16_tflops_sustained", peak)),
                "frac_of_datasheet_peak": tflops_per_gpu / DATASHEET_BF16_TFLOPS}
    if use_split and shared_tile:
        # decoding: one pass over K and V is the whole cost; the roof is HBM, not the tensor core
        hbm = float(peaks["hbm_gbs"])
        gbs = touched / (ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": f"attn_fwd_kernel (split-KV, {n_chunks} chunks, heads of a KV group share a tile) + fwd_merge_kernel",
                    "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm, "peak_kind": f"{peak_kind} copy bandwidth",
                    "traffic": NCU_TRAFFIC_BYTES.get(cfg.name), "algorithmic_bytes": int(touched)}
    elif use_split:
        roofline["kernel"] = f"attn_fwd_kernel (split-KV, {n_chunks} chunks) + fwd_merge_kernel"
    line = {
        "metric": f"fused attention {'fwd+bwd' if with_bwd else 'fwd'} TFLOP/s ({'fp16' if f16 else 'bf16'})", "value": value, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": paper_ratio(cfg.name, mode, ms) if world == 1 and not f16 else None,
        "dtype": args.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "B_per_gpu": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "Sq": cfg.Sq, "Sk": cfg.Sk,
                   "D": cfg.D, "causal": cfg.causal, "mode": mode, "l2": l2_note, "splitkv_chunks": n_chunks if use_split else None,
                   "launch": "cuda graph replay of one step" if args.graph else "library calls",
                   "flops_convention": "4*B*Hq*Sq*Sk*D fwd (x0.5 causal), bwd = 2.5x fwd",
                   "parallelism": f"dp{world} (batch shards, no collective)"},
        "pct_of_measured_bf16_peak": 100.0 * tflops_per_gpu / peak,
        "pct_of_datasheet_bf16_peak": 100.0 * tflops_per_gpu / DATASHEET_BF16_TFLOPS,
        "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline,
    }
    if NCU_TRAFFIC_NOTE.get(cfg.name):
        roofline["traffic_note"] = NCU_TRAFFIC_NOTE[cfg.name]
    for key, val in extras.items():
        if world > 1:
            val = dict(val, value=val["value"] * world, note=f"whole job: {world} ranks, each the same per-GPU work")
        line[key] = val
    if world == 1 and not args.no_cpu_baseline and not args.lean:
        line["cpu_baseline"] = cpu_baseline(cfg, with_bwd, budget_s=args.cpu_budget)
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# the oracle as the CPU baseline / reference arm
# ----------------------------------------------------------------------------------------------
def _oracle_sample(cfg, with_bwd, heads, rows):
    """Oracle inputs for `heads` KV groups of batch 0 and the first `rows` query rows.  For a
    non-causal workload any row subset is an exact sub-workload; for a causal one the first rows
    form a causal problem of their own (keys beyond them are invisible)."""
    from oracle import attn_oracle as orc
    G = cfg.Hq // cfg.Hkv
    if int(cfg.causal) == 1:
        sk = rows                                   # top-left aligned: the first rows see only the first keys
    elif int(cfg.causal) == 2:
        sk = max(1, rows + cfg.Sk - cfg.Sq)         # bottom-right aligned: same offset between last query and last key
    else:
        sk = cfg.Sk
    sub = cfg.with_(B=1, Hq=heads * G, Hkv=heads, Sq=rows, Sk=sk)
    bits = make_inputs(sub, with_do=with_bwd)
    return orc, sub, bits


def _oracle_step(orc, sub, bits, with_bwd):
    t0 = time.perf_counter()
    orc.attn_fwd(bits[0], bits[1], bits[2], sub.causal, sub.scale)
    if with_bwd:
        orc.attn_bwd(bits[0], bits[1], bits[2], bits[3], sub.causal, sub.scale)
    return time.perf_counter() - t0


def _rows_for_budget(cfg, with_bwd, heads, rate_flops_per_s, budget_s, floor_rows):
    """Query rows whose oracle time is about budget_s at the probed rate (flops by the benchmark's convention)."""
    mult = 3.5 if with_bwd else 1.0
    hq = heads * (cfg.Hq // cfg.Hkv)
    target = budget_s * rate_flops_per_s
    if int(cfg.causal) == 1:          # sub-problem is rows x rows, causal: 2 * hq * rows^2 * D * mult flops
        rows = (target / (2.0 * hq * cfg.D * mult)) ** 0.5
    else:                   # rows x Sk: 4 * hq * rows * Sk * D * mult flops
        rows = target / (4.0 * hq * cfg.Sk * cfg.D * mult)
    return int(max(floor_rows, min(cfg.Sq, rows)))


def _probe_rate(cfg, with_bwd, heads, probe_rows):
    o, sub, bits = _oracle_sample(cfg, with_bwd, heads, probe_rows)
    _oracle_step(o, sub, bits, with_bwd)                       # warm-up (thread pool, page faults)
    t = _oracle_step(o, sub, bits, with_bwd)
    return sub.fwd_flops() * (3.5 if with_bwd else 1.0) / max(t, 1e-9)


def cpu_baseline(cfg, with_bwd, budget_s=15.0):
    from oracle import attn_oracle as orc
    cores = orc.num_threads()
    heads = min(cfg.Hkv * cfg.B, cores)
    probe_rows = min(cfg.Sq, 256)
    rate = _probe_rate(cfg, with_bwd, heads, probe_rows)
    rows = _rows_for_budget(cfg, with_bwd, heads, rate, budget_s, probe_rows)
    o, sub, bits = _oracle_sample(cfg, with_bwd, heads, rows)
    t = _oracle_step(o, sub, bits, with_bwd)
    flops = sub.fwd_flops() * (3.5 if with_bwd else 1.0)
    return {"value": flops / t / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "seconds": t,
            "sample": f"{heads} KV groups x first {rows} query rows of {cfg.name} "
                      f"({'fwd+bwd' if with_bwd else 'fwd'}, fp64, {flops / 1e9:.1f} GFLOP by the same convention)"}


def run_reference(args):
    rank, _, world = env_rank_world()
    if rank != 0:
        return
    if args.workload in VARLEN_CONFIGS or args.workload == "decode_ragged":
        raise SystemExit("--impl reference covers the fixed-length workloads; packed ones report the oracle as cpu_baseline")
    if args.workload in RING_WORKLOADS:          # the oracle knows no ranks: the whole causal sequence, forward + backward
        from paper_2601_16238_b200.inputs import AttnConfig
        w = RING_WORKLOADS[args.workload]
        cfg = AttnConfig(args.workload, w["index"], w["B"], w["Hq"], w["Hkv"], w["S"], w["S"], w["D"], True, True)
        args.mode = "fwd_bwd"
    else:
        cfg = CONFIGS[args.workload]
    mode = args.mode or "fwd"
    with_bwd = mode == "fwd_bwd"
    from oracle import attn_oracle as orc
    cores = orc.num_threads()
    heads = min(cfg.Hkv * cfg.B, cores)
    total = args.steps + args.warmup
    per_step_budget = max(0.05, args.ref_budget / max(total, 1))
    probe_rows = min(cfg.Sq, 128)
    rate = _probe_rate(cfg, with_bwd, heads, probe_rows)
    rows = _rows_for_budget(cfg, with_bwd, heads, rate, per_step_budget, min(cfg.Sq, 16))
    o, sub, bits = _oracle_sample(cfg, with_bwd, heads, rows)
    for _ in range(args.warmup):
        _oracle_step(o, sub, bits, with_bwd)
    times = [_oracle_step(o, sub, bits, with_bwd) for _ in range(args.steps)]
    sec = float(np.mean(times))
    flops = sub.fwd_flops() * (3.5 if with_bwd else 1.0)
    value = flops / sec / 1e12
    sample = (f"each step: {heads} KV groups x first {rows} query rows of {cfg.name}, "
              f"{'fwd+bwd' if with_bwd else 'fwd'}, fp64 ({flops / 1e9:.2f} GFLOP by the same convention)")
    line = {
        "impl": "reference", "metric": f"fused attention {'fwd+bwd' if with_bwd else 'fwd'} TFLOP/s (bf16)",
        "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": cfg.name, "B_per_gpu": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "Sq": cfg.Sq, "Sk": cfg.Sk,
                   "D": cfg.D, "causal": cfg.causal, "mode": mode},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# Kernel-suite workloads: the other rows of the paper's kernel microbenchmark table, at its shapes.
# They are bound by HBM bandwidth, so the metric is the bandwidth the algorithmic bytes are moved at.
# ------------------------------------------------------------------------------------------------
SUITE_WORKLOADS = {
    # name: (shape, the paper's best latency on its H100 PCIe in ms, kernels launched per step)
    "rmsnorm_fwd": ((4096, 8192), 0.13, 1),
    "layernorm_fwd_bwd": ((4096, 8192), 0.45, 3),
    "rope_fwd": ((4, 8, 2048, 128), 0.14, 1),
    # named in the paper's description of the suite, without a table row: shapes chosen here
    "softmax_fwd": ((8192, 8192), None, 1),
    "cross_entropy_fwd_bwd": ((8192, 32768), None, 1),
    "adamw_step": ((1 << 26,), None, 1),
}
SUITE_EPS = 1e-5


def _suite_inputs(name, shape):
    """Seeded bf16 bit patterns: x (and dy) ~ N(0, 1), weights 1 + N(0, 1) / 4, bias N(0, 1) / 2."""
    from paper_2601_16238_b200.inputs import f32_to_bf16_bits, normal_bf16
    if name in ("rope_fwd", "softmax_fwd", "cross_entropy_fwd_bwd"):
        return {"x": normal_bf16(shape, 7001)}
    if name == "adamw_step":
        return {"g": normal_bf16(shape, 7001)}
    cols = shape[1]
    wide = lambda s: (normal_bf16((cols,), s).astype(np.uint32) << np.uint32(16)).view(np.float32)
    return {"x": normal_bf16(shape, 7001), "dy": normal_bf16(shape, 7002), "w": f32_to_bf16_bits(1.0 + 0.25 * wide(7003)),
            "b": f32_to_bf16_bits(0.5 * wide(7004))}


def _suite_bytes(name, shape):
    n = int(np.prod(shape)) * 2
    if name == "rmsnorm_fwd":
        return 2 * n + shape[1] * 2                       # x in, y out, w
    if name == "layernorm_fwd_bwd":
        return 5 * n + shape[0] * 16 + shape[1] * 14      # fwd: x, y; bwd: x, dy, dx; mean / rstd written and read; w, b, dw, db
    if name == "softmax_fwd":
        return 2 * n
    if name == "cross_entropy_fwd_bwd":
        return 2 * n + shape[0] * 16                      # the fused kernel: logits in, dlogits out, per-row scalars
    if name == "adamw_step":
        return shape[0] * 26                              # p, m, v (fp32) read and written, g (bf16) read
    return 2 * n + shape[2] * shape[3] * 4                # x in, y out, the cos / sin tables


def _suite_oracle_step(name, ins, rows):
    """One oracle pass over the first `rows` rows (rotary: heads) of the workload; returns the rows it covered."""
    from oracle import suite_oracle as so
    if name == "rope_fwd":
        x = so.bf16_bits_to_f64(ins["x"].reshape(-1, *ins["x"].shape[2:])[:rows])
        cos, sin = so.rope_tables(x.shape[1], x.shape[2])
        so.rope_apply(x, cos, sin)
        return x.shape[0]
    if name == "adamw_step":
        g = so.bf16_bits_to_f64(ins["g"][:rows])
        so.adamw_step(np.zeros(rows), g, np.zeros(rows), np.zeros(rows), 1, 1e-3, 0.9, 0.95, 1e-8, 0.1)
        return rows
    if name == "softmax_fwd":
        so.softmax_fwd(so.bf16_bits_to_f64(ins["x"][:rows]))
        return rows
    if name == "cross_entropy_fwd_bwd":
        x = so.bf16_bits_to_f64(ins["x"][:rows])
        t = np.arange(rows) % x.shape[1]
        so.cross_entropy_fwd(x, t)
        so.cross_entropy_bwd(x, t, np.ones(rows))
        return rows
    x, w = so.bf16_bits_to_f64(ins["x"][:rows]), so.bf16_bits_to_f64(ins["w"])
    if name == "rmsnorm_fwd":
        so.rmsnorm_fwd(x, w, SUITE_EPS)
    else:
        so.layernorm_fwd(x, w, so.bf16_bits_to_f64(ins["b"]), SUITE_EPS)
        so.layernorm_bwd(x, w, so.bf16_bits_to_f64(ins["dy"][:rows]), SUITE_EPS)
    return x.shape[0]


def _suite_cpu_baseline(name, shape, ins, budget_s):
    total_rows = shape[0] if name != "rope_fwd" else shape[0] * shape[1]      # (adamw_step: elements)
    rows = max(1, total_rows // 64)
    t0 = time.perf_counter(); _suite_oracle_step(name, ins, rows); dt = time.perf_counter() - t0
    rows = int(min(total_rows, max(rows, rows * budget_s / max(dt, 1e-6) / 2)))
    t0 = time.perf_counter(); done = _suite_oracle_step(name, ins, rows); dt = time.perf_counter() - t0
    gbs = _suite_bytes(name, shape) * (done / total_rows) / dt / 1e9
    return {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"{done} of {total_rows} rows in {dt:.2f} s (numpy float64, one thread)"}


def run_suite(args):
    name = args.workload
    shape, paper_ms, launches = SUITE_WORKLOADS[name]
    ins = _suite_inputs(name, shape)
    nbytes = _suite_bytes(name, shape)
    rank, local_rank, world = env_rank_world()
    if args.impl == "reference":
        if rank != 0:
            return
        t_all = time.perf_counter()
        base = _suite_cpu_baseline(name, shape, ins, min(args.cpu_budget, args.ref_budget / max(1, args.steps + args.warmup)))
        line = {"impl": "reference", "metric": "effective_bandwidth", "value": base["value"], "unit": "GB/s", "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": nbytes / base["value"] / 1e6, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": name, "shape": list(shape)}, "cpu_baseline": base,
                "e2e": {"value": base["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0,
                "wall_s": time.perf_counter() - t_all}
        print(json.dumps(line), flush=True)
        return
    import torch
    from paper_2601_16238_b200 import suite
    torch.cuda.set_device(local_rank)
    init_process_group("nccl")
    peaks, peak_kind = load_peaks()
    t = {k: torch.from_numpy(v.view(np.int16)).view(torch.bfloat16).cuda() for k, v in ins.items()}
    # L2 is flushed by READING a buffer twice its size: a write flush would leave the cache full of dirty lines whose
    # write-back lands in the timed kernel, which matters for kernels that run at HBM speed for ~25 us
    flush_buf = torch.zeros(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.max()
    if name == "rmsnorm_fwd":
        y = torch.empty_like(t["x"])
        step = lambda: suite.vt_suite_rmsnorm_fwd(t["x"], t["w"], SUITE_EPS, y)
        result = y
    elif name == "layernorm_fwd_bwd":
        rows, cols = shape
        y, dx = torch.empty_like(t["x"]), torch.empty_like(t["x"])
        mean, rstd = torch.empty(rows, device="cuda"), torch.empty(rows, device="cuda")
        dw, db = torch.empty(cols, device="cuda"), torch.empty(cols, device="cuda")
        ws = torch.empty(suite.vt_suite_layernorm_bwd_workspace_bytes(cols), dtype=torch.uint8, device="cuda")
        def step():
            suite.vt_suite_layernorm_fwd(t["x"], t["w"], t["b"], SUITE_EPS, y, mean, rstd)
            suite.vt_suite_layernorm_bwd(t["x"], t["w"], t["dy"], mean, rstd, dx, dw, db, ws)
        result = dx
    elif name == "softmax_fwd":
        y = torch.empty_like(t["x"])
        step = lambda: suite.vt_suite_softmax_fwd(t["x"], y)
        result = y
    elif name == "cross_entropy_fwd_bwd":
        rows, cols = shape
        tgt = (torch.arange(rows, device="cuda", dtype=torch.int32) * 7919) % cols
        loss, lse = torch.empty(rows, device="cuda"), torch.empty(rows, device="cuda")
        dl = torch.full((rows,), 1.0 / rows, device="cuda")
        dx = torch.empty_like(t["x"])
        step = lambda: suite.vt_suite_cross_entropy_fwd_bwd(t["x"], tgt, dl, loss, lse, dx)      # one pass: logits in, gradient out
        result = loss
    elif name == "adamw_step":
        n = shape[0]
        pp, mm, vv = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        step = lambda: suite.vt_suite_adamw_step(pp, t["g"], mm, vv, 1, 1e-3, 0.9, 0.95, 1e-8, 0.1)
        result = pp[:1 << 20]
    else:
        cos, sin = suite.vt_suite_rope_tables(shape[2], shape[3])
        y = torch.empty_like(t["x"])
        step = lambda: suite.vt_suite_rope_apply(t["x"], cos, sin, False, y)
        result = y
    with ClockSampler(local_rank) as clocks:
        ms = max_over_ranks(time_steps(torch, step, args.steps, args.warmup, flush), device="cuda")
    # end to end: the inputs start in pinned host memory and the main result returns there, every step
    host_in = {k: v.cpu().pin_memory() for k, v in t.items()}
    host_out = torch.empty_like(result, device="cpu").pin_memory()
    def e2e_step():
        for k in t:
            t[k].copy_(host_in[k], non_blocking=True)
        step()
        host_out.copy_(result, non_blocking=True)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms = max_over_ranks(time_steps(torch, e2e_step, e2e_steps, 3), device="cuda")
    if rank != 0:
        return
    gbs = nbytes / (ms * 1e-3) / 1e9
    h2d = sum(v.numel() * v.element_size() for v in t.values())
    d2h = result.numel() * result.element_size()
    line = {"metric": "effective_bandwidth", "value": gbs * world, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": (paper_ms / ms) if (paper_ms and world == 1) else None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": name, "shape": list(shape), "io": "bf16", "l2": "flushed between iterations (252 MB read)",
                       "replicas": world},
            "roofline": {"bound": "hbm", "kernel": name, "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                         "frac": gbs / float(peaks["hbm_gbs"]), "peak_kind": f"{peak_kind} copy bandwidth", "traffic": None,
                         "algorithmic_bytes": int(nbytes)},
            "paper_context": {"paper_best_ms_h100_pcie": paper_ms, "ours_ms": ms, "ratio": paper_ms / ms} if paper_ms else None,
            "e2e": {"value": nbytes * world / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": launches * args.steps, "clocks": clocks.summary()}
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = _suite_cpu_baseline(name, shape, ins, args.cpu_budget)
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="sdpa_s8192_nc", choices=sorted(CONFIGS) + sorted(VARLEN_CONFIGS) + sorted(SUITE_WORKLOADS) + sorted(RING_WORKLOADS) + ["decode_ragged"])
    ap.add_argument("--mode", choices=["fwd", "fwd_bwd"], default=None)
    ap.add_argument("--splitkv", choices=["auto", "on", "off"], default="auto",
                    help="forward through vt_attn_fwd_splitkv: auto = when the library's plan splits the keys or packs a KV group's heads")
    ap.add_argument("--dtype", choices=["bf16", "f16"], default="bf16",
                    help="element type of the tensors (the metric is stated in bf16; f16 runs the *_f16 entry points, fixed-length workloads only)")
    ap.add_argument("--graph", action="store_true",
                    help="time replays of a CUDA graph holding one step's kernels (small workloads: takes the host's per-call work out)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--lean", action="store_true",
                    help="only the timed region: no end-to-end leg, no forward+backward / sustained extras, no CPU baseline (the "
                         "command line profiler captures run)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work for the cpu_baseline object")
    ap.add_argument("--ref-budget", type=float, default=150.0, help="seconds the whole --impl reference run may take")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.workload in SUITE_WORKLOADS:
        run_suite(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
