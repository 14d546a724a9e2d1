#!/usr/bin/env python
"""Benchmark of the graded decode-attention hot path.

A step = one decode step of the whole hot path over all layers of the workload:
per layer, gkv_append_demote (append one token per sequence, close/demote blocks) followed by
gkv_decode_attn over the graded cache (config 3 adds gkv_quest_select and reads the selected
pages).  Metric: effective context tokens/s = batch * context / step time, plus achieved HBM GB/s
of the decode kernel against the measured copy bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

N > 1 runs N independent replicas (the path has no exchange step), one process per GPU under
torchrun; `value` sums the replicas' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_23599_b200 import workloads as W  # noqa: E402

METRIC = "graded decode-attn effective ctx tokens/s and HBM GB/s as % of 8 TB/s roofline"
UNIT = "ctx tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum of one decode_kernel launch from an ncu capture
# (profiles/ holds the summary); None = not captured for that workload.
DRAM_TRAFFIC_PER_LAUNCH = {"cfg2_llama8b_append": 335.9e6}    # 330.1 MB read + 5.8 MB written (ncu, one launch)


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled during the timed region."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return res


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return rank, local, world


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, world: int) -> float:
    """Replicas do not exchange data; the only collective is this maximum of the per-rank times
    (NCCL on the GPUs; the CPU tests run it over gloo)."""
    if world == 1:
        return x
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(world: int, batch: int, ctx: int, ms_step: float) -> float:
    """Whole-job context tokens/s of `world` replicas whose slowest rank took ms_step per step."""
    return world * batch * ctx / (ms_step * 1e-3)


# --------------------------------------------------------------------------------------------------
def build_cache(w: W.Workload, n_layers: int, extra_ctx: int, device):
    """Generate each layer on the GPU, ingest it, free it."""
    from paper_2608_23599_b200 import binding as B
    import dataclasses
    wl = dataclasses.replace(w, max_ctx=w.ctx + extra_ctx, n_layers=n_layers)
    cache = B.Cache(B.config_from_workload(wl, n_layers), device=device)
    qs = []
    ingest_ms, in_bytes = [], 0
    for layer in range(n_layers):
        data = W.make_layer(wl, layer, device)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cache.gkv_append_demote(layer, data["k"], data.get("v"), token_mass=data.get("mass"))
        e1.record()
        torch.cuda.synchronize()
        ingest_ms.append(e0.elapsed_time(e1))
        in_bytes = data["k"].numel() * 2 + (data["v"].numel() * 2 if data.get("v") is not None else 0)
        qs.append(data["q"])
        del data
    # the prompt's bulk ingest (one gkv_append_demote call per layer: statistics, level plan, every block
    # encoded once at its planned level), outside the timed decode region; the first layer also pays
    # for first-use set-up, so the median is reported
    med = sorted(ingest_ms)[(len(ingest_ms) - 1) // 2]
    ingest = {"ms_per_layer_call_median": med, "ms_first_layer_call": ingest_ms[0],
              "prompt_tokens_per_s": wl.batch * wl.ctx / (med * 1e-3),
              "input_GBs": in_bytes / (med * 1e-3) / 1e9, "input_bytes_per_layer_call": in_bytes}
    return wl, cache, qs, ingest


def run_ours(args, rank, local, world):
    from paper_2608_23599_b200 import binding as B
    B.build()
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    w = W.config(args.config)
    n_layers = args.layers or w.n_layers
    K, Wm = args.steps, args.warmup
    total_steps = 2 * (K + Wm) + 8
    wl, cache, q0, ingest = build_cache(w, n_layers, total_steps + 64, device)
    Bsz, Hq, Hkv, d, dv = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.d_k, wl.d_v
    alias = bool(wl.v_aliases_k)
    gen = torch.Generator(device=device)
    gen.manual_seed(4242 + rank)
    # per-step decode inputs, resident in HBM for the device-timed region
    k_new = torch.randn((total_steps, n_layers, Bsz, 1, Hkv, d), generator=gen, device=device).to(torch.bfloat16)
    v_new = None if alias else torch.randn((total_steps, n_layers, Bsz, 1, Hkv, dv), generator=gen, device=device).to(torch.bfloat16)
    q_new = torch.randn((total_steps, n_layers, Bsz, Hq, d), generator=gen, device=device).to(torch.bfloat16)
    out = torch.empty((n_layers, Bsz, Hq, dv), dtype=torch.float32, device=device)
    quest = wl.page_tokens > 0 and wl.quest_budget_tokens > 0
    k_sel = wl.quest_budget_tokens // wl.page_tokens if quest else 0
    pages = torch.zeros((Bsz, Hkv, max(k_sel, 1)), dtype=torch.int32, device=device) if quest else None

    # The loops below hand the library plain device addresses (worked out once, here) instead of a
    # fresh tensor view per call, as a serving loop in C++ would: on the small workloads the per-call
    # host time would otherwise be the bound.  The buffers are the tensors above.
    cache.stream_handle = torch.cuda.current_stream().cuda_stream
    k_stride, v_stride, q_stride, o_stride = Bsz * Hkv * d * 2, Bsz * Hkv * dv * 2, Bsz * Hq * d * 2, Bsz * Hq * dv * 4
    k_at = lambda s_, l_: k_new.data_ptr() + (s_ * n_layers + l_) * k_stride
    v_at = (lambda s_, l_: None) if alias else (lambda s_, l_: v_new.data_ptr() + (s_ * n_layers + l_) * v_stride)
    q_at = lambda s_, l_: q_new.data_ptr() + (s_ * n_layers + l_) * q_stride
    out_at = [out.data_ptr() + l_ * o_stride for l_ in range(n_layers)]
    pages_at = pages.data_ptr() if quest else None
    budget = wl.quest_budget_tokens

    def step_device(s):
        for l in range(n_layers):
            cache.gkv_append_demote(l, k_at(s, l), v_at(s, l), n_new=1)
            if quest:
                n_sel = cache.gkv_quest_select(l, q_at(s, l), budget, pages_at)
                cache.gkv_decode_attn(l, q_at(s, l), out_at[l], page_idx=pages_at, n_sel=n_sel)
            else:
                cache.gkv_decode_attn(l, q_at(s, l), out_at[l])

    # ---- device-resident timing -------------------------------------------------------------------
    s = 0
    for _ in range(Wm):
        step_device(s)
        s += 1
    ctx_start = cache.gkv_ctx_len(0)
    sampler = ClockSampler(local)
    barrier(world)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    closes = 0
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(K)]      # end of every step (per-step times)
    fill_steps = []
    for i in range(K):
        step_device(s)
        s += 1
        marks[i].record()
        if cache.gkv_ctx_len(0) % 64 == 0:
            closes += 1
            fill_steps.append(i)
    ev1.record()
    barrier(world)
    clocks = sampler.stop()
    ms_step = max_over_ranks(ev0.elapsed_time(ev1) / K, world)
    per_step = [(ev0 if i == 0 else marks[i - 1]).elapsed_time(marks[i]) for i in range(K)]
    plain = sorted(t for i, t in enumerate(per_step) if i not in fill_steps)
    step_detail = {"ms_median_step_without_block_fill": plain[len(plain) // 2] if plain else None,
                   "ms_block_fill_steps": [per_step[i] for i in fill_steps]}
    value = aggregate_value(world, Bsz, ctx_start, ms_step)

    # ---- dominant kernel: decode_attn alone, per launch -------------------------------------------
    rep = cache.gkv_bits_report(0)
    algo_bytes = rep.last_read_bits / 8 + Bsz * Hq * d * 2 + Bsz * Hq * dv * 4
    if quest:
        algo_bytes = (rep.last_read_bits - rep.box_bits) / 8 + Bsz * Hq * d * 6
    reps = max(3, min(20, int(2e10 / max(algo_bytes * n_layers, 1))))
    for l in range(n_layers):
        if quest:
            cache.gkv_decode_attn(l, q_at(0, l), out_at[l], page_idx=pages_at, n_sel=k_sel)
        else:
            cache.gkv_decode_attn(l, q_at(0, l), out_at[l])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for r in range(reps):
        for l in range(n_layers):
            if quest:
                cache.gkv_decode_attn(l, q_at(r % total_steps, l), out_at[l], page_idx=pages_at, n_sel=k_sel)
            else:
                cache.gkv_decode_attn(l, q_at(r % total_steps, l), out_at[l])
    e1.record()
    torch.cuda.synchronize()
    us_launch = e0.elapsed_time(e1) * 1e3 / (reps * n_layers)
    # the same call on one layer back to back: its bytes stay in the 126 MB L2 when they fit (labelled warm)
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record()
    for r in range(20):
        if quest:
            cache.gkv_decode_attn(0, q_at(r % total_steps, 0), out_at[0], page_idx=pages_at, n_sel=k_sel)
        else:
            cache.gkv_decode_attn(0, q_at(r % total_steps, 0), out_at[0])
    w1.record()
    torch.cuda.synchronize()
    us_launch_one_layer = w0.elapsed_time(w1) * 1e3 / 20
    achieved = algo_bytes / (us_launch * 1e-6) / 1e9
    peak, peak_kind = measured_hbm_peak()
    traffic = DRAM_TRAFFIC_PER_LAUNCH.get(wl.name)
    scorer = None
    if quest:
        # the page scorer on its own (score + top-k launches): it reads every box of the layer
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for r in range(reps):
            for l in range(n_layers):
                cache.gkv_quest_select(l, q_at(r % total_steps, l), budget, pages_at)
        s1.record()
        torch.cuda.synchronize()
        us_sel = s0.elapsed_time(s1) * 1e3 / (reps * n_layers)
        scorer = {"us_per_call": us_sel, "box_bytes_per_call": rep.box_bits / 8,
                  "achieved": rep.box_bits / 8 / (us_sel * 1e-6) / 1e9, "unit": "GB/s"}

    # ---- end to end: host buffers, H2D of the step's inputs and D2H of its result inside the region
    # One pinned record per layer: [new keys | new values | queries].  Layer 0's record goes up on the
    # compute stream; the other layers' records go up on a second stream while layer 0 computes (one event
    # wait before layer 1).  The outputs of all layers but the last come back on the second stream while
    # the last layer computes; the last layer's output follows on the compute stream.  The caller then waits
    # for both streams: every byte of the step's inputs and outputs crosses PCIe inside the timed region.
    k_el, v_el, q_el = Bsz * Hkv * d, (0 if alias else Bsz * Hkv * dv), Bsz * Hq * d
    rec = k_el + v_el + q_el
    hin = torch.randn((n_layers, rec)).to(torch.bfloat16).pin_memory()
    din = torch.empty_like(hin, device=device)
    hout = torch.empty((n_layers, Bsz, Hq, dv), dtype=torch.float32).pin_memory()
    dk_at = [din.data_ptr() + l_ * rec * 2 for l_ in range(n_layers)]
    dv_at = [None if alias else dk_at[l_] + k_el * 2 for l_ in range(n_layers)]
    dq_at = [dk_at[l_] + (k_el + v_el) * 2 for l_ in range(n_layers)]
    main_stream = torch.cuda.current_stream()
    side = torch.cuda.Stream(device=device)
    ev_in, ev_mid = torch.cuda.Event(), torch.cuda.Event()

    def layer_e2e(l):
        cache.gkv_append_demote(l, dk_at[l], dv_at[l], n_new=1)
        if quest:
            n_sel = cache.gkv_quest_select(l, dq_at[l], budget, pages_at)
            cache.gkv_decode_attn(l, dq_at[l], out_at[l], page_idx=pages_at, n_sel=n_sel)
        else:
            cache.gkv_decode_attn(l, dq_at[l], out_at[l])

    def step_e2e():
        din[0:1].copy_(hin[0:1], non_blocking=True)
        if n_layers > 1:
            with torch.cuda.stream(side):
                din[1:].copy_(hin[1:], non_blocking=True)
                ev_in.record(side)
        layer_e2e(0)
        if n_layers > 1:
            main_stream.wait_event(ev_in)
            for l in range(1, n_layers - 1):
                layer_e2e(l)
            ev_mid.record(main_stream)
            with torch.cuda.stream(side):
                side.wait_event(ev_mid)
                hout[:n_layers - 1].copy_(out[:n_layers - 1], non_blocking=True)
            layer_e2e(n_layers - 1)
        hout[n_layers - 1:].copy_(out[n_layers - 1:], non_blocking=True)
        main_stream.synchronize()                      # the caller consumes the step's result
        if n_layers > 1:
            side.synchronize()

    for _ in range(Wm):
        step_e2e()
    ctx_e2e = cache.gkv_ctx_len(0)
    barrier(world)
    t0 = time.perf_counter()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(K):
        step_e2e()
    g1.record()
    barrier(world)
    wall_ms = (time.perf_counter() - t0) * 1e3 / K
    e2e_ms = max_over_ranks(g0.elapsed_time(g1) / K, world)
    e2e_value = world * Bsz * ctx_e2e / (e2e_ms * 1e-3)
    h2d = hin.numel() * 2
    d2h = hout.numel() * 4

    launches_per_layer = 2 + (2 if quest else 0)      # append, decode with fused merge (+ score, top-k)
    # a block close adds the block-statistics kernel and, under the staircase policy, one encode launch
    gpu_launches = K * n_layers * launches_per_layer + closes * n_layers * ((0 if alias else 1) + (1 if wl.policy == W.POLICY_STAIRCASE else 0))

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16",       # tensor-core operands; f32 accumulation
        "dtype_detail": "bf16 exact rows / int8-int4-int2 codes dequantised to f16 operands, f32 accumulate",
        "data": "synthetic",
        "config": {"workload": wl.name, "batch": Bsz, "context": ctx_start, "n_layers": n_layers,
                   "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": d, "resident_bpv": rep.bpv_resident,
                   "l2": "inputs larger than L2: each layer call streams %.0f MB" % (algo_bytes / 1e6),
                   "parallelism": "replicas x%d" % world, "block_fills_in_timed_region": closes},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"]},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms, "host_wall_ms_per_step": wall_ms},
        "gpu_launches": gpu_launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_kind": peak_kind + " copy bandwidth",
                     "kernel": "decode_kernel (split-K partials merged in the same launch; timed per gkv_decode_attn call)",
                     "us_per_launch": us_launch, "algorithmic_bytes_per_launch": algo_bytes,
                     "us_per_launch_same_layer_back_to_back": us_launch_one_layer,
                     "same_layer_fits_l2": bool(algo_bytes < 100e6),
                     "frac_of_8TBs": achieved / NOMINAL_HBM_GBS},
        "ctx_tokens_per_s_per_layer_call": Bsz * ctx_start / (us_launch * 1e-6),
        # gkv_append_demote next to gkv_decode_attn: what a layer's append adds to its decode call in a
        # plain step, and the steps in which a block fills (close, demotions, new work lists)
        "append_demote": {"us_per_layer_in_plain_step": max(0.0, (step_detail["ms_median_step_without_block_fill"] or ms_step) * 1e3 / n_layers
                                                             - us_launch - (scorer["us_per_call"] if scorer else 0.0)),
                          **step_detail},
    }
    line["bulk_ingest"] = ingest
    if rank == 0 and wl.config_id == 1 and n_layers > 1:
        line["all_layers_in_one_launch"] = one_launch_figure(wl, n_layers, device)
    if scorer:
        line["quest_select"] = scorer
    if rank == 0:
        line["cpu_baseline"] = cpu_baseline(wl, n_layers, budget_s=args.cpu_seconds)
    cache.close()
    return line


# --------------------------------------------------------------------------------------------------
def one_launch_figure(w: W.Workload, n_layers: int, device):
    """Config 1 reads ~5 MB per layer call and is bound by launch latency.  For scale: the same amount of
    cache as all layers of a step, laid out as n_layers sequences of ONE layer, read by ONE decode launch.
    This is not a model step (a layer's query depends on the layer before it); it shows what the kernel
    does with the step's bytes when they come in one launch."""
    from paper_2608_23599_b200 import binding as B
    import dataclasses
    wide = dataclasses.replace(w, batch=w.batch * n_layers, n_layers=1)
    cache = B.Cache(B.config_from_workload(wide, 1), device=device)
    data = W.make_layer(wide, 0, device)
    cache.gkv_append_demote(0, data["k"], data.get("v"), token_mass=data.get("mass"))
    q = data["q"]
    out = torch.empty((wide.batch, wide.n_q_heads, wide.d_v), dtype=torch.float32, device=device)
    for _ in range(3):
        cache.gkv_decode_attn(0, q, out)
    torch.cuda.synchronize()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)      # larger than the 126 MB L2
    times = []
    for _ in range(10):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cache.gkv_decode_attn(0, q, out)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    rep = cache.gkv_bits_report(0)
    nbytes = rep.last_read_bits / 8 + q.numel() * 2 + out.numel() * 4
    us = sorted(times)[len(times) // 2]
    cache.close()
    return {"us": us, "bytes": nbytes, "GB/s": nbytes / (us * 1e-6) / 1e9, "sequences": wide.batch,
            "l2": "flushed before every launch",
            "note": "n_layers x batch sequences of one layer in one launch; not a model step"}


# --------------------------------------------------------------------------------------------------
def cpu_baseline(w: W.Workload, n_layers: int, budget_s: float = 20.0, steps: int = 1):
    """The oracle as it stands, timed on the host cores on a bounded sample: S streams of one layer
    (ingest untimed), one decode step = append one token + graded attention; scaled to the whole
    workload (all streams, all layers)."""
    import dataclasses
    from oracle import gkv_oracle as O
    S = 1
    ctx_scale = 1
    if w.ctx > 131072:
        # a million-token stream takes the numpy oracle minutes: time a 1/16 context with the same
        # ladder proportions and scale linearly (the oracle's cost is linear in the context)
        ctx_scale = 16
        w = dataclasses.replace(w, ctx=w.ctx // ctx_scale, max_ctx=w.ctx // ctx_scale + 128,
                                stair_tokens=tuple((t // ctx_scale) // 64 * 64 for t in w.stair_tokens))
    ws = dataclasses.replace(w, batch=1, n_kv_heads=S, n_q_heads=S * w.group_size, n_layers=1)
    data = W.make_layer(ws, 0, "cpu")
    cfg = O.Config(n_layers=1, batch=1, n_q_heads=ws.n_q_heads, n_kv_heads=S, d_k=w.d_k, d_v=w.d_v,
                   v_aliases_k=w.v_aliases_k, page_tokens=w.page_tokens, policy=w.policy, stair_tokens=tuple(w.stair_tokens),
                   n_sink_blocks=w.n_sink_blocks, retire_after=w.retire_after, rd_budget_bpv=w.rd_budget_bpv,
                   residual_fraction=w.residual_fraction, softmax_scale=w.softmax_scale)
    oc = O.GradedCache(cfg)
    f32 = lambda t: t.to(torch.float32).numpy()
    mass = data.get("mass")
    oc.append_demote(0, f32(data["k"]), None if data.get("v") is None else f32(data["v"]),
                     token_mass=None if mass is None else mass.numpy())
    times = []
    t_begin = time.perf_counter()
    i = 0
    while i < max(1, steps) or (time.perf_counter() - t_begin < budget_s and i < 8):
        tok = W.make_decode_tokens(ws, 0, i, "cpu")
        kk, vv, qq = f32(tok["k"]), (None if tok["v"] is None else f32(tok["v"])), f32(tok["q"])
        t0 = time.perf_counter()
        oc.append_demote(0, kk, vv)
        if w.page_tokens > 0 and w.quest_budget_tokens > 0:
            sel = oc.quest_select(0, qq, w.quest_budget_tokens)
            oc.decode_attn(0, qq, sel)
        else:
            oc.decode_attn(0, qq)
        times.append(time.perf_counter() - t0)
        i += 1
    t_stream = float(np.median(times))
    n_streams = w.batch * w.n_kv_heads
    t_step = t_stream * n_streams / S * n_layers * ctx_scale
    return {"value": w.batch * w.ctx * ctx_scale / t_step, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
            "sample": "%d of %d streams of 1 of %d layers%s, %d decode steps (append + attention), median, "
                      "scaled linearly to all streams and layers" % (S, n_streams, n_layers,
                                                                      " at 1/%d of the context" % ctx_scale if ctx_scale > 1 else "",
                                                                      len(times)),
            "seconds_per_stream_step": t_stream}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    w = W.config(args.config)
    n_layers = args.layers or w.n_layers
    t0 = time.perf_counter()
    base = cpu_baseline(w, n_layers, budget_s=0.0, steps=args.warmup + args.steps)
    ms = (time.perf_counter() - t0) * 1e3
    return {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": w.batch * w.ctx / base["value"] * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "context": w.ctx, "n_layers": n_layers},
            "cpu_baseline": {"value": base["value"], "unit": UNIT, "cores": base["cores"], "kind": "oracle",
                             "sample": base["sample"]},
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_ms_total": ms}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload: 0..4 (default 2: Llama-8B-like batched decode); 5 = RD-V2 operating point")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (0 = as defined)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        world = int(os.environ.get("WORLD_SIZE", "1"))
        line = run_reference(args, rank, world)
        if line is not None:
            print(json.dumps(line))
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local, world = dist_setup(args.gpus)
    line = run_ours(args, rank, local, world)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
