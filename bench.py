#!/usr/bin/env python
"""Benchmark of the GPTAQ per-layer solve on B200.

One step = one pass of the whole hot path over one synthetic layer:
reset -> accumulate (all token batches) -> factor -> build_P -> quantize.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2]
    python bench.py --impl reference ...     # the float64 CPU oracle, bounded sample

Prints ONE JSON line (rank 0).  With N > 1 (launched by torchrun) the ranks
share ONE layer: every rank accumulates its share of the token batches, one
all-reduce sums H and dXX^T, every rank factors and then quantizes its slab
of the rows of W (strong scaling; the value is the time of that one layer).
``--replicas`` instead gives every rank an independent layer of the same
shape (no data-path collective; the value is the time per layer of the job).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "ms per layer (GPTAQ solve: accumulate + factor + P + quantize)"

# dram__bytes_read.sum + dram__bytes_write.sum of one stats_umma_kernel launch (one token batch) from an
# ncu capture of the kernel as it stands, keyed by (workload, statistics arithmetic); workloads without a
# capture of the current kernel report null with the reason.
STATS_KERNEL_TRAFFIC = {("cfg2", 0): 462.5e6}
TRAFFIC_MISSING = "no ncu capture of the current statistics kernel for this workload and arithmetic"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.stop, self.th = index, [], threading.Event(), None

    def _run(self):
        while not self.stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.rows.append([c.strip() for c in out.strip().split(",")])
            except Exception:
                pass
            self.stop.wait(0.1)

    def __enter__(self):
        self.th = threading.Thread(target=self._run, daemon=True)
        self.th.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        self.th.join(timeout=6)

    def summary(self):
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg: wl.LayerConfig, sample_tokens: int, sample_rows: int):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload and scales to the whole
    layer: statistics are linear in tokens, rows of W are independent.  Beyond n = 4096 the sample shrinks so
    that it stays near 10-30 s of CPU work (fewer tokens and rows), and beyond n = 16384 -- where a float64
    factorisation of the whole n x n matrix takes hours -- factor, P and the loop run on the leading 8192
    input channels and are scaled by the cubes / squares of the width ratio.  Returns (ms per layer,
    description, threads)."""
    from oracle import gptaq_oracle as orc
    threads = torch.get_num_threads()
    n_s = cfg.n if cfg.n <= 16384 else 8192
    shrink = min(1.0, 4096.0 / n_s)
    sample_tokens = min(max(256, int(sample_tokens * shrink)), cfg.batch_tokens)
    sample_rows = min(max(8, int(sample_rows * shrink * shrink)), cfg.m)
    X, Xfp = (t.numpy()[:, :n_s] for t in wl.make_batch(cfg, 0, "cpu", sample_tokens))
    W = wl.make_weight(cfg, "cpu", rows=sample_rows).numpy()[:, :n_s]
    st = orc.new_stats(n_s)
    t0 = time.perf_counter()
    orc.accumulate(st, X, Xfp)
    t_acc = time.perf_counter() - t0
    t0 = time.perf_counter()
    sample_damp = max(cfg.damp, 0.05)                            # few tokens: keep the sample SPD
    U, dead = orc.factor(st.H, st.tokens, sample_damp)
    t_fac = time.perf_counter() - t0
    t0 = time.perf_counter()
    P = orc.build_P(st.D, st.tokens, U, cfg.alpha)
    t_p = time.perf_counter() - t0
    t0 = time.perf_counter()
    orc.quantize(W, U, P, dead, cfg.bits, cfg.group, cfg.sym)
    t_q = time.perf_counter() - t0
    w = cfg.n / n_s                                              # width ratio of the layer to the sample
    total = t_acc * (cfg.tokens / sample_tokens) * w * w + (t_fac + t_p) * w ** 3 + t_q * (cfg.m / sample_rows) * w * w
    width = "" if n_s == cfg.n else (f"; all of it on the leading {n_s} of {cfg.n} input channels, statistics and loop scaled "
                                     f"by the width ratio squared, factor and P by its cube")
    desc = (f"accumulate on {sample_tokens} of {cfg.tokens} tokens ({t_acc:.2f} s, scaled by tokens); "
            f"factor ({t_fac:.2f} s; damp raised from {cfg.damp} to {sample_damp} so that the sample's H, from fewer "
            f"tokens than input channels, stays positive definite) and P ({t_p:.2f} s) in full; column loop on "
            f"{sample_rows} of {cfg.m} rows ({t_q:.2f} s, scaled by rows){width}")
    return total * 1e3, desc, threads


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    desc, threads = "", 0
    for i in range(args.warmup + args.steps):
        ms, desc, threads = oracle_sample(cfg, args.ref_tokens, args.ref_rows)
        if i >= args.warmup:
            times.append(ms)
    v = sum(times) / len(times)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": "ms", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(wl.describe(cfg), parallelism="cpu oracle, rank 0 only"),
        "cpu_baseline": {"value": v, "unit": "ms", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- multi-rank plumbing
def rank_config(cfg: wl.LayerConfig, rank: int) -> wl.LayerConfig:
    """Every rank solves its own layer of the same shape: same recipe, seed shifted by the rank."""
    return wl.scaled(cfg, seed=cfg.seed + rank)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Largest per-rank time (one all-reduce of a scalar; the only collective, outside the timed region)."""
    if world <= 1:
        return ms
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def per_layer_ms(ms_step: float, world: int) -> float:
    """One step solves `world` independent layers at once: time per layer of the whole job."""
    return ms_step / world


# --------------------------------------------------------------------------- CUDA leg
def run_ours(args, cfg):
    import paper_2504_02692_b200 as g
    from paper_2504_02692_b200 import build as gbuild
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        # the communicator's own log lines (ranks, transport) stay on: they are the record of what the
        # all-reduce ran over
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        gbuild.build()
    if world > 1:
        dist.barrier()
    g.load_library()
    pk = peaks()

    # inputs resident in HBM before the timed region (each rank its own layer: seed = rank)
    shard = (world > 1 and not args.replicas) or args.shard_layer
    if shard:
        # ONE layer across the ranks: this rank's share of the token batches and of the rows of W
        from paper_2504_02692_b200 import sharded
        if world > 1 and cfg.n_batches < world:
            raise SystemExit(f"{cfg.n_batches} token batches cannot be shared by {world} ranks")
        cfg_r = cfg
        my_batches = sharded.token_shard(cfg.n_batches, rank, world)
        r0, r1 = sharded.row_shard(cfg.m, rank, world)
        batches = [wl.make_batch(cfg_r, b, dev) for b in my_batches]
        W0 = wl.make_weight(cfg_r, dev)[r0:r1].contiguous()
        cfg = wl.scaled(cfg, m=r1 - r0)
    else:
        cfg_r = rank_config(cfg, rank)
        batches = [wl.make_batch(cfg_r, b, dev) for b in range(cfg.n_batches)]
        W0 = wl.make_weight(cfg_r, dev)
    if cfg.w_bf16:
        W0 = W0.to(torch.bfloat16)
    G = 1 if cfg.group <= 0 else (cfg.n + cfg.group - 1) // cfg.group
    codes = torch.empty((cfg.m, cfg.n), dtype=torch.uint8, device=dev)
    scales = torch.empty((cfg.m, G), dtype=torch.float32, device=dev)
    zeros = torch.empty((cfg.m, G), dtype=torch.float32, device=dev)
    Wq = torch.empty((cfg.m, cfg.n), dtype=torch.float32, device=dev)
    # statistics arithmetic: the cheapest tensor-core mode that keeps U within its error bound
    st = g.LayerState(cfg.n, cfg.m, cfg.batch_tokens, cfg.blocksize, dev, total_tokens=args.full_tokens)
    h = st.handle
    prec = g.gptaq_recommended_stats_precision(cfg.n, args.full_tokens)
    if args.full_split_statistics:
        prec = g.GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR
    prec_name = {g.GPTAQ_STATS_FP16_TENSOR: "fp16 operands, fp32 accumulate",
                 g.GPTAQ_STATS_FP16_SPLIT_TENSOR: "fp16 hi+lo split for H, fp32 accumulate",
                 g.GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR: "fp16 hi+lo split for H and dXX^T, fp32 accumulate"}[prec]
    stream = torch.cuda.current_stream()
    if args.full_split_statistics:
        g.gptaq_set_stats_precision(h, prec)
    if args.act_order:
        g.gptaq_set_act_order(h, True)
    if args.clip_search > 0:
        g.gptaq_set_clip_search(h, args.clip_search, 0.2)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(marks=None):
        g.gptaq_reset(h)
        e0 = ev(); e0.record(stream)
        for X, Xfp in batches:
            g.gptaq_accumulate(h, X, Xfp)
        if shard:
            sharded.allreduce_statistics(st)     # the one exchange step: sum of H and dXX^T over the ranks
        g.gptaq_flush(h)            # the products run on the handle's own stream: order `stream` after them
        e1 = ev(); e1.record(stream)
        g.gptaq_factor(h, cfg.damp)
        e2 = ev(); e2.record(stream)
        g.gptaq_build_P(h, cfg.alpha)
        e3 = ev(); e3.record(stream)
        g.gptaq_quantize(h, W0, cfg.bits, cfg.group, cfg.sym, cfg.blocksize, codes, scales, zeros, Wq)
        e4 = ev(); e4.record(stream)
        if marks is not None:
            marks.append((e0, e1, e2, e3, e4))

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    status = g.gptaq_sync_status(h)
    if status[0] != g.GPTAQ_OK:
        raise RuntimeError(f"device status {status}")

    marks = []
    sync_all()
    g.gptaq_set_kernel_timing(h, True)       # event pairs around the statistics kernel on its own stream
    g.gptaq_stats_kernel_time(h)
    l0 = g.gptaq_launch_count(h)
    t_beg, t_end = ev(), ev()
    with ClockSampler(local) as clk:
        t_beg.record(stream)
        for _ in range(args.steps):
            step(marks)
        t_end.record(stream)
        sync_all()
    launches = g.gptaq_launch_count(h) - l0
    kern_ms_total, kern_launches = g.gptaq_stats_kernel_time(h)
    g.gptaq_set_kernel_timing(h, False)
    ms_total = t_beg.elapsed_time(t_end)
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    ms_layer = ms_step if shard else per_layer_ms(ms_step, world)

    acc_step_ms = sum(m[0].elapsed_time(m[1]) for m in marks) / args.steps
    acc_call_ms = acc_step_ms / max(1, len(batches))      # conversion and product of consecutive batches overlap
    fac_ms = sum(m[1].elapsed_time(m[2]) for m in marks) / args.steps
    p_ms = sum(m[2].elapsed_time(m[3]) for m in marks) / args.steps
    q_ms = sum(m[3].elapsed_time(m[4]) for m in marks) / args.steps
    # algorithmic flops of one accumulate call: the upper triangle of H (n^2 k) and what P needs of dXX^T:
    # the part above the diagonal (n^2 k), or all of it under act_order (2 n^2 k)
    flops_per_token = (3.0 if args.act_order else 2.0) * cfg.n * cfg.n
    flops_call = flops_per_token * cfg.batch_tokens
    stage_achieved = flops_call / (acc_call_ms * 1e-3) / 1e12     # whole accumulate call: conversion, product, fix-up
    peak = pk["bf16_sustained"]
    if kern_launches > 0:
        # the dominant kernel by itself: algorithmic flops of the timed region / the sum of its launch durations
        kern_us = kern_ms_total * 1e3 / kern_launches
        flops_launch = flops_per_token * cfg.batch_tokens * len(batches) * args.steps / kern_launches
        achieved = flops_launch / (kern_us * 1e-6) / 1e12
        kern_name = "stats_umma_kernel (tcgen05 kind::f16, cta_group::2), one token batch per launch"
    else:
        # small widths accumulate on the float32 FMA kernel: the stage is the unit
        kern_us, flops_launch, achieved = acc_call_ms * 1e3, flops_call, stage_achieved
        kern_name = "gptaq_accumulate (one token batch; float32 FMA path of small widths)"

    # end to end through the host entry points: pinned host buffers in, host results out
    e2e = None
    if not args.no_e2e:
        hb = [(X.cpu().pin_memory(), Xfp.cpu().pin_memory()) for X, Xfp in batches]
        hW = (W0.float() if cfg.w_bf16 else W0).cpu().pin_memory()
        hcodes = torch.empty((cfg.m, cfg.n), dtype=torch.uint8).pin_memory()
        hs = torch.empty((cfg.m, G), dtype=torch.float32).pin_memory()
        hz = torch.empty((cfg.m, G), dtype=torch.float32).pin_memory()
        stage = torch.empty(max(2 * cfg.batch_tokens * cfg.n * 4, g.gptaq_quantize_stage_bytes(cfg.m, cfg.n, cfg.group)),
                            dtype=torch.uint8, device=dev)

        def step_host():
            g.gptaq_reset(h)
            for X, Xfp in hb:
                g.gptaq_accumulate_host(h, X, Xfp, stage)
            if shard:
                sharded.allreduce_statistics(st)
            g.gptaq_factor(h, cfg.damp)
            g.gptaq_build_P(h, cfg.alpha)
            g.gptaq_quantize_host(h, hW, cfg.bits, cfg.group, cfg.sym, cfg.blocksize, hcodes, hs, hz, stage)

        step_host()
        sync_all()
        a, b = ev(), ev()
        a.record(stream)
        ke = max(1, min(args.steps, 3))
        for _ in range(ke):
            step_host()
        b.record(stream)
        sync_all()
        ems = a.elapsed_time(b) / ke
        ems = max_over_ranks(ems, world, dev)
        h2d = sum(x.numel() * 4 * 2 for x, _ in hb) + hW.numel() * 4
        d2h = hcodes.numel() + (hs.numel() + hz.numel()) * 4
        e2e = {"value": ems if shard else per_layer_ms(ems, world), "unit": "ms", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    if rank != 0:
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, desc, threads = oracle_sample(cfg, args.ref_tokens, args.ref_rows)
        cpu = {"value": v, "unit": "ms", "cores": threads, "kind": "oracle", "sample": desc}
    # Per-stage rooflines (algorithmic work / stage time against the bound that applies): the products of
    # factor, P and the lazy-batch update run as three tensor-core products on split operands: fp16 hi / lo
    # parts where the width is a multiple of 8 (at most bf16 peak / 3 of useful flops), TF32 parts otherwise
    # (bf16 peak / 2 / 3); the column loop is bound by HBM on paper.
    fp16_split = cfg.n >= 512 and cfg.n % 8 == 0
    split_peak = peak / 3.0 if fp16_split else peak / 2.0 / 3.0
    split_name = "tensor (3xFP16 split)" if fp16_split else "tensor (3xTF32)"
    n_, m_, B_ = float(cfg.n), float(cfg.m), float(cfg.blocksize)
    fl_factor, fl_P = 2.0 * n_ ** 3 / 3.0, 2.0 * n_ ** 3 / 3.0
    fl_trail = 2.0 * m_ * n_ * n_ * max(0.0, 1.0 - B_ / n_)
    by_loop = 25.0 * m_ * n_ + 8.0 * n_ * B_
    layer_roofline_ms = (flops_call * len(batches) / (peak * 1e12) + (fl_factor + fl_P + fl_trail) / (split_peak * 1e12)
                         + by_loop / (pk["hbm_gbs"] * 1e9)) * 1e3
    stage_rooflines = {
        "factor": {"bound": split_name, "achieved": fl_factor / (fac_ms * 1e-3) / 1e12, "peak": split_peak, "unit": "TFLOP/s"},
        "build_P": {"bound": split_name, "achieved": fl_P / (p_ms * 1e-3) / 1e12, "peak": split_peak, "unit": "TFLOP/s"},
        "quantize": {"bound": split_name + " + hbm", "trailing_update_tflops_if_alone": fl_trail / (q_ms * 1e-3) / 1e12,
                     "column_loop_gbs_if_alone": by_loop / (q_ms * 1e-3) / 1e9, "peak_tflops": split_peak,
                     "peak_gbs": pk["hbm_gbs"]},
        "layer": {"roofline_ms": layer_roofline_ms, "measured_ms": ms_step, "frac": layer_roofline_ms / ms_step},
    }
    for k in ("factor", "build_P"):
        stage_rooflines[k]["frac"] = stage_rooflines[k]["achieved"] / split_peak
    line = {
        "metric": METRIC, "value": ms_layer, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False, "scaling": "strong" if shard else "weak",
        "vs_baseline": None, "dtype": "f16 x f16 -> f32 (statistics), f32 (solve; its products as 3 x f16 hi/lo -> f32)", "data": "synthetic",
        "config": dict(wl.describe(cfg), parallelism=(f"one layer over {world} GPUs: tokens sharded, one all-reduce of H and dXX^T, rows sharded"
                                    if shard else f"{world} independent layer(s), one per GPU"),
                       l2="inputs (%.1f GB per step) exceed L2" % (2 * cfg.tokens * cfg.n * 4 / 1e9),
                       statistics=prec_name, act_order=bool(args.act_order), clip_search=args.clip_search,
                       dxx="all of it (act_order permutes it)" if args.act_order else "above the diagonal (what P uses)"),
        "stages_ms": {"accumulate": acc_step_ms, "factor": fac_ms, "build_P": p_ms, "quantize": q_ms,
                      "layer_quantize": fac_ms + p_ms + q_ms},
        "accumulate_tflops": stage_achieved, "stage_rooflines": stage_rooflines,
        "roofline": {"kernel": kern_name, "bound": "tensor", "achieved": achieved,
                     "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "kernel_us_per_launch": kern_us, "kernel_launches": kern_launches,
                     "accumulate_stage": {"what": "whole gptaq_accumulate call (conversion prologue + product + fix-up)",
                                          "us_per_batch": acc_call_ms * 1e3, "achieved": stage_achieved,
                                          "frac": stage_achieved / peak, "frac_of_burst": stage_achieved / pk["bf16_burst"]},
                     "traffic": STATS_KERNEL_TRAFFIC.get((cfg.name, prec)),
                     "traffic_note": None if (cfg.name, prec) in STATS_KERNEL_TRAFFIC else TRAFFIC_MISSING,
                     "peak_source": pk["source"] + " bf16 cuBLAS, sustained (the accumulate stage runs for "
                                    "milliseconds under the power cap)",
                     "peak_burst": pk["bf16_burst"], "frac_of_burst": achieved / pk["bf16_burst"],
                     "algorithmic_flops_per_launch": flops_launch},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clk.summary(),
    }
    if args.batches > 0:
        line["truncated"] = f"{cfg.n_batches} token batches only: not a benchmark value"
    print(json.dumps(line), flush=True)


def run_p_rowwise(args):
    """Latency of P in its two forms (Theorem 4.2 as two matrix products vs. Eq. "unparallel" row by row),
    the comparison of the paper's Section 5 ("Efficiency"), on synthetic layers of width 1024 and 4096."""
    import paper_2504_02692_b200 as g
    from paper_2504_02692_b200 import build as gbuild
    torch.cuda.set_device(0)
    gbuild.build()
    g.load_library()
    stream = torch.cuda.current_stream()
    out = {}
    for n in (1024, 4096):
        cfg = wl.scaled(wl.CONFIGS["cfg2"], name=f"p{n}", n=n, m=128, n_batches=2)
        batches = [wl.make_batch(cfg, b, "cuda") for b in range(cfg.n_batches)]
        st = g.LayerState(cfg.n, cfg.m, cfg.batch_tokens, cfg.blocksize, "cuda", total_tokens=cfg.tokens)
        h = st.handle
        times = {"theorem_4_2": [], "row_by_row": []}
        for name, fn in (("theorem_4_2", g.gptaq_build_P), ("row_by_row", g.gptaq_build_P_rowwise)):
            for i in range(args.warmup + args.steps):
                g.gptaq_reset(h)
                for X, Xfp in batches:
                    g.gptaq_accumulate(h, X, Xfp)
                g.gptaq_factor(h, cfg.damp)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn(h, cfg.alpha)
                e1.record(stream)
                torch.cuda.synchronize()
                if i >= args.warmup:
                    times[name].append(e0.elapsed_time(e1))
        status = g.gptaq_sync_status(h)
        if status[0] != g.GPTAQ_OK:
            raise RuntimeError(f"device status {status}")
        med = {k: sorted(v)[len(v) // 2] for k, v in times.items()}
        out[f"n{n}"] = {"theorem_4_2_ms": med["theorem_4_2"], "row_by_row_ms": med["row_by_row"],
                        "ratio": med["row_by_row"] / med["theorem_4_2"]}
        st.close()
    print(json.dumps({"metric": "ms to build P, two forms (includes the operand copies for the loop)", "unit": "ms",
                      "steps": args.steps, "warmup": args.warmup, "p_rowwise": out, "data": "synthetic",
                      "truncated": "comparison of two forms of one stage: not a benchmark value"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--ref-tokens", type=int, default=8192)
    ap.add_argument("--ref-rows", type=int, default=None,
                    help="rows of W in the oracle's timed sample (default: 512 for the cpu_baseline leg of a GPU run, 128 per "
                         "step of --impl reference, so that 25 steps stay near two minutes)")
    ap.add_argument("--batches", type=int, default=0,
                    help="profiler captures only: keep this many token batches (the line is marked truncated)")
    ap.add_argument("--replicas", action="store_true",
                    help="N > 1: one independent layer per rank (weak scaling, no collective) instead of the default, "
                         "one layer across the ranks (token-sharded statistics, one all-reduce, row-sharded quantize)")
    ap.add_argument("--shard-layer", action="store_true",
                    help="the default for N > 1; at N = 1 it forces the same code path with one rank holding every shard "
                         "(the all-reduce is a no-op), as a check of that path on one GPU")
    ap.add_argument("--clip-search", type=int, default=0,
                    help="clipping-range search of the grids with this many candidates (off in the headline configuration)")
    ap.add_argument("--act-order", action="store_true", help="columns sorted by diag(H) (off in the headline configuration)")
    ap.add_argument("--full-split-statistics", action="store_true",
                    help="both statistics with split fp16 operands (float32-grade, 3x the MMAs; off in the headline configuration)")
    ap.add_argument("--p-rowwise", action="store_true",
                    help="times P as two matrix products (Theorem 4.2) against the row-by-row form at n = 1024 and 4096 "
                         "and prints that comparison instead of the benchmark line")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.workload]
    full_tokens = cfg.tokens
    if args.batches > 0:
        cfg = wl.scaled(cfg, n_batches=min(args.batches, cfg.n_batches))
    args.full_tokens = full_tokens
    if args.ref_rows is None:
        args.ref_rows = 128 if args.impl == "reference" else 512
    if args.impl == "reference":
        run_reference(args, cfg)
    elif args.p_rowwise:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py --p-rowwise needs a CUDA device")
        run_p_rowwise(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); "
                             "use --impl reference for the CPU oracle")
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
