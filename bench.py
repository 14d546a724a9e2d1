#!/usr/bin/env python
"""Benchmark of the graded decode-attention hot path.

A step = one decode step of the whole hot path over all layers of the workload:
per layer, gkv_append_demote (append one token per sequence, close/demote blocks) followed by
gkv_decode_attn over the graded cache (config 3 adds gkv_quest_select and reads the selected
pages).  Metric: effective context tokens/s = batch * context / step time, plus achieved HBM GB/s
of the decode kernel against the measured copy bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

The prompt is ingested a few tokens short of the workload's context so that the context reaches it -
and a block of every stream fills: close, box / statistics kernels, demotions, new work lists - in
the middle of the timed region.  After the headline workload the other workloads run briefly in the
same process and are printed in the `per_config` block (rank 0, one GPU).

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

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the workload's dominant kernel from an ncu
# capture (profiles/ holds the summaries); None = not captured for that workload.
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (ncu captures
# summarised under profiles/): config 2 330.0 MB read + 3.8 MB written, config 4 386.4 + 6.7 MB
DRAM_TRAFFIC_PER_LAUNCH = {"cfg2_llama8b_append": 333.8e6, "cfg4_mla_1m": 382.3e6}


def dominant_kernel(w) -> str:
    if w.v_aliases_k:
        return "mla_decode_kernel + mla_combine_kernel (timed per gkv_decode_attn call)"
    if w.page_tokens > 0 and w.quest_budget_tokens > 0:
        return "decode_kernel<page list> (split-K partials merged in the same launch; timed per gkv_decode_attn call)"
    return "decode_kernel (split-K partials merged in the same launch; timed per gkv_decode_attn call)"


def ingest_context(ctx: int, steps: int, warmup: int) -> int:
    """Tokens to ingest so that the context reaches `ctx` (a multiple of 64: a block of every stream
    fills) at the middle step of the timed region."""
    return ctx - (warmup + steps // 2 + 1) % 64


def config_dict(w, n_layers: int, ctx_start: int, world: int) -> dict:
    """Description of the workload: the same keys and values in both arms."""
    return {"workload": w.name, "batch": w.batch, "context": ctx_start, "n_layers": n_layers, "n_q_heads": w.n_q_heads,
            "n_kv_heads": w.n_kv_heads, "head_dim": w.d_k, "l2": "inputs larger than L2: consecutive layer calls stream distinct caches",
            "parallelism": "replicas x%d" % world}


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
def build_cache(w: W.Workload, n_layers: int, extra_ctx: int, device, ctx_ingest=None):
    """Generate each layer on the GPU, ingest it, free it."""
    from paper_2608_23599_b200 import binding as B
    import dataclasses
    wl = dataclasses.replace(w, ctx=w.ctx if ctx_ingest is None else ctx_ingest, max_ctx=w.ctx + extra_ctx, n_layers=n_layers)
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


def measure(w, n_layers, K, Wm, rank, local, world, cpu_seconds, full=True):
    """One workload: device-resident steps, the decode call on its own, (full) end to end with host
    buffers and the CPU baseline.  Returns the JSON line of the workload."""
    from paper_2608_23599_b200 import binding as B
    device = torch.device("cuda", local)
    total_steps = 2 * (K + Wm) + 8
    wl, cache, q0, ingest = build_cache(w, n_layers, total_steps + 64, device, ingest_context(w.ctx, K, Wm))
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
    ms_sorted = sorted(per_step)
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

    e2e = None
    if full:
        e2e = measure_e2e(cache, wl, n_layers, K, Wm, world, device, out, out_at, pages_at, quest, budget, alias)
    launches_per_layer = 2 + (2 if quest else 0) + (1 if alias else 0)      # append, decode with fused merge (+ score, top-k; + combine)
    # a block close adds the block-statistics kernel and, under the staircase policy, one encode launch
    gpu_launches = K * n_layers * launches_per_layer + closes * n_layers * ((0 if alias else 1) + (1 if wl.policy == W.POLICY_STAIRCASE else 0))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_step, "ms_per_step_median": ms_sorted[len(ms_sorted) // 2], "ms_per_step_min": ms_sorted[0],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16",       # tensor-core operands (exact integers and hi + lo pairs); f32 accumulation
        "dtype_detail": "bf16 exact rows / int8-int4-int2 codes as exact f16 integers, scaled operands as f16 hi + lo pairs, f32 accumulate",
        "data": "synthetic",
        "config": config_dict(w, n_layers, ctx_start, world),
        "workload_state": {"resident_bpv": rep.bpv_resident, "bpv_paper": rep.bpv_paper, "block_fills_in_timed_region": closes,
                           "MB_streamed_per_layer_call": algo_bytes / 1e6},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"]},
        "gpu_launches": gpu_launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_kind": peak_kind + " copy bandwidth",
                     "kernel": dominant_kernel(wl),
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
    if e2e:
        line["e2e"] = e2e
    line["bulk_ingest"] = ingest
    if full and rank == 0 and wl.config_id == 1 and n_layers > 1:
        line["all_layers_in_one_launch"] = one_launch_figure(w, n_layers, device)
    if scorer:
        line["quest_select"] = scorer
    if rank == 0:
        line["parity_sample"] = parity_sample(w)
    if full and rank == 0:
        line["cpu_baseline"] = cpu_baseline(w, n_layers, ctx_start, budget_s=cpu_seconds)
    cache.close()
    del cache, k_new, v_new, q_new, out
    torch.cuda.empty_cache()
    return line


def measure_e2e(cache, wl, n_layers, K, Wm, world, device, out, out_at, pages_at, quest, budget, alias):
    Bsz, Hq, Hkv, d, dv = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.d_k, wl.d_v
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
    return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": e2e_ms, "host_wall_ms_per_step": wall_ms}


# --------------------------------------------------------------------------------------------------
# Which layer counts / step counts the brief per-config runs use (the headline workload runs as defined).
BRIEF = {0: dict(layers=1, steps=12, warmup=3), 1: dict(layers=36, steps=8, warmup=3), 2: dict(layers=4, steps=8, warmup=3),
         3: dict(layers=4, steps=8, warmup=3), 4: dict(layers=2, steps=6, warmup=3), 5: dict(layers=4, steps=8, warmup=3),
         6: dict(layers=4, steps=8, warmup=3)}


def run_ours(args, rank, local, world):
    from paper_2608_23599_b200 import binding as B
    B.build()
    torch.cuda.set_device(torch.device("cuda", local))
    w = W.config(args.config)
    n_layers = args.layers or w.n_layers
    line = measure(w, n_layers, args.steps, args.warmup, rank, local, world, args.cpu_seconds, full=True)
    if rank == 0 and world == 1 and not args.no_per_config:
        per = {}
        for cid in (0, 1, 2, 3, 4, 5, 6):
            if cid == args.config:
                continue
            wc = W.config(cid)
            b = BRIEF[cid]
            m = measure(wc, min(b["layers"], wc.n_layers), b["steps"], b["warmup"], rank, local, world, 0.0, full=False)
            entry = {"workload": wc.name, "n_layers_run": m["config"]["n_layers"], "n_layers_of_workload": wc.n_layers,
                     "context": m["config"]["context"], "us_per_call": m["roofline"]["us_per_launch"],
                     "algorithmic_bytes": m["roofline"]["algorithmic_bytes_per_launch"], "GBs": m["roofline"]["achieved"],
                     "frac": m["roofline"]["frac"], "kernel": m["roofline"]["kernel"],
                     "ms_per_step_of_layers_run": m["ms_per_step"],
                     "ms_per_step_median_of_layers_run": m["ms_per_step_median"],
                     "ms_per_step_scaled_to_workload": m["ms_per_step"] * wc.n_layers / m["config"]["n_layers"],
                     "ms_per_step_median_scaled_to_workload": m["ms_per_step_median"] * wc.n_layers / m["config"]["n_layers"],
                     # the median over the steps that close no block (the medians above count every step)
                     "ms_plain_step_median_scaled_to_workload": (m["append_demote"]["ms_median_step_without_block_fill"] or m["ms_per_step_median"])
                     * wc.n_layers / m["config"]["n_layers"],
                     "resident_bpv": m["workload_state"]["resident_bpv"], "bpv_paper": m["workload_state"]["bpv_paper"],
                     "block_fills_in_timed_region": m["workload_state"]["block_fills_in_timed_region"],
                     "ms_block_fill_steps": m["append_demote"]["ms_block_fill_steps"],
                     "parity_sample": m.get("parity_sample")}
            if "quest_select" in m:
                entry["quest_select"] = m["quest_select"]
            per["config_%d" % cid] = entry
        line["per_config"] = per
    return line


def parity_sample(w: W.Workload):
    """Largest output error of one sampled stream against the oracle (checker use): the stream is ingested
    and read once by both sides.  Million-token streams are sampled at 1/16 of the context with the same
    ladder proportions (the oracle needs minutes for the full length)."""
    import dataclasses
    from oracle import gkv_oracle as O
    from paper_2608_23599_b200 import binding as B
    scale = 16 if w.ctx > 131072 else 1
    ws = dataclasses.replace(w, batch=1, n_kv_heads=1, n_q_heads=w.group_size, n_layers=1, ctx=w.ctx // scale,
                             max_ctx=w.ctx // scale + 128,
                             stair_tokens=tuple(t if t < 0 else (t // scale) // 64 * 64 for t in w.stair_tokens))
    data = W.make_layer(ws, 0, "cpu")
    cfg = O.Config(n_layers=1, batch=1, n_q_heads=ws.n_q_heads, n_kv_heads=1, d_k=w.d_k, d_v=w.d_v, v_aliases_k=w.v_aliases_k,
                   max_ctx=ws.max_ctx, page_tokens=w.page_tokens, policy=w.policy, stair_tokens=tuple(ws.stair_tokens),
                   n_sink_blocks=w.n_sink_blocks, retire_after=w.retire_after, rd_budget_bpv=w.rd_budget_bpv,
                   residual_fraction=w.residual_fraction, quest_reduce=w.quest_reduce, softmax_scale=w.softmax_scale)
    oc = O.GradedCache(cfg)
    f32 = lambda t: None if t is None else t.to(torch.float32).numpy()
    mass = data.get("mass")
    oc.append_demote(0, f32(data["k"]), f32(data.get("v")), token_mass=None if mass is None else mass.numpy())
    gc = B.Cache(B.config_from_workload(ws, 1))
    dev = gc.device
    gc.gkv_append_demote(0, data["k"].to(dev), None if data.get("v") is None else data["v"].to(dev),
                         token_mass=None if mass is None else mass.to(dev).contiguous())
    out = torch.empty((1, ws.n_q_heads, w.d_v), dtype=torch.float32, device=dev)
    q = data["q"]
    if w.page_tokens > 0 and w.quest_budget_tokens > 0:
        k = w.quest_budget_tokens // w.page_tokens
        pages = torch.zeros((1, 1, k), dtype=torch.int32, device=dev)
        n_sel = gc.gkv_quest_select(0, q.to(dev), w.quest_budget_tokens, pages)
        gc.gkv_decode_attn(0, q.to(dev), out, page_idx=pages, n_sel=n_sel)
        sel = oc.quest_select(0, f32(q), w.quest_budget_tokens)
        torch.cuda.synchronize()
        pages_equal = bool(np.array_equal(pages.cpu().numpy()[0, 0, :n_sel], sel[0][0]))
        ref, _ = oc.decode_attn(0, f32(q), sel)
    else:
        gc.gkv_decode_attn(0, q.to(dev), out)
        torch.cuda.synchronize()
        pages_equal = None
        ref, _ = oc.decode_attn(0, f32(q))
    got = out.cpu().numpy().astype(np.float64)
    err = float(np.abs(got - ref).max())
    rel = float((np.linalg.norm(got - ref, axis=-1) / (np.linalg.norm(ref, axis=-1) + 1e-30)).max())
    levels_equal = bool(np.array_equal(gc.gkv_debug_export_levels(0, 0, 0), oc.levels(0, 0, 0)))
    gc.close()
    res = {"max_abs_error": err, "relative_l2": rel, "levels_equal": levels_equal, "bound": "2e-3 / 1e-2",
           "sample": "one stream of one layer%s, ingest + one read, against the CPU oracle" % (" at 1/16 of the context" if scale > 1 else "")}
    if pages_equal is not None:
        res["selected_pages_equal"] = pages_equal
    return res


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
def cpu_baseline(w: W.Workload, n_layers: int, ctx_start: int, budget_s: float = 20.0, steps: int = 1):
    """The oracle as it stands, timed on the host cores on a bounded sample: one stream of one layer
    (ingest of ctx_start tokens untimed), one decode step = append one token + graded attention (+ page
    selection).  `seconds_per_stream_step` is what was timed; `value` scales it linearly to the whole
    workload (all streams, all layers).  The oracle is plain numpy: its loops run on one thread, its
    matrix products on however many threads the BLAS library takes - `threads_used` is the process CPU
    time over the wall time of the timed steps, and `value_1_thread` repeats the sample with the
    library pools limited to one thread."""
    import dataclasses
    from oracle import gkv_oracle as O
    S = 1
    ctx_scale = 1
    ctx = ctx_start
    if w.ctx > 131072:
        # a million-token stream takes the numpy oracle minutes: time a 1/16 context with the same
        # ladder proportions and scale linearly (the oracle's cost is linear in the context)
        ctx_scale = 16
        ctx = ctx_start // ctx_scale
        w = dataclasses.replace(w, stair_tokens=tuple(t if t < 0 else (t // ctx_scale) // 64 * 64 for t in w.stair_tokens))
    ws = dataclasses.replace(w, batch=1, n_kv_heads=S, n_q_heads=S * w.group_size, n_layers=1, ctx=ctx, max_ctx=ctx + 256)
    data = W.make_layer(ws, 0, "cpu")
    cfg = O.Config(n_layers=1, batch=1, n_q_heads=ws.n_q_heads, n_kv_heads=S, d_k=w.d_k, d_v=w.d_v,
                   v_aliases_k=w.v_aliases_k, max_ctx=ws.max_ctx, page_tokens=w.page_tokens, policy=w.policy,
                   stair_tokens=tuple(w.stair_tokens), n_sink_blocks=w.n_sink_blocks, retire_after=w.retire_after,
                   rd_budget_bpv=w.rd_budget_bpv, residual_fraction=w.residual_fraction, quest_reduce=w.quest_reduce,
                   softmax_scale=w.softmax_scale)
    oc = O.GradedCache(cfg)
    f32 = lambda t: t.to(torch.float32).numpy()
    mass = data.get("mass")
    oc.append_demote(0, f32(data["k"]), None if data.get("v") is None else f32(data["v"]),
                     token_mass=None if mass is None else mass.numpy())
    step_no = [0]

    def one_step():
        tok = W.make_decode_tokens(ws, 0, step_no[0], "cpu")
        step_no[0] += 1
        kk, vv, qq = f32(tok["k"]), (None if tok["v"] is None else f32(tok["v"])), f32(tok["q"])
        t0 = time.perf_counter()
        oc.append_demote(0, kk, vv)
        if w.page_tokens > 0 and w.quest_budget_tokens > 0:
            sel = oc.quest_select(0, qq, w.quest_budget_tokens)
            oc.decode_attn(0, qq, sel)
        else:
            oc.decode_attn(0, qq)
        return time.perf_counter() - t0

    times = []
    t_begin = time.perf_counter()
    cpu0 = time.process_time()
    while len(times) < max(1, steps) or (time.perf_counter() - t_begin < budget_s and len(times) < 8):
        times.append(one_step())
    threads_used = (time.process_time() - cpu0) / max(time.perf_counter() - t_begin, 1e-9)
    t_stream = float(np.median(times))
    t_one = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            torch_threads = torch.get_num_threads()
            torch.set_num_threads(1)
            t_one = float(np.median([one_step() for _ in range(max(1, min(3, len(times))))]))
            torch.set_num_threads(torch_threads)
    except Exception:
        t_one = None
    n_streams = w.batch * w.n_kv_heads
    scale = n_streams / S * n_layers * ctx_scale
    value = lambda t: w.batch * ctx_start / (t * scale)
    res = {"value": value(t_stream), "unit": UNIT, "cores": max(1, int(round(threads_used))), "threads_used": threads_used,
           "cores_available": len(os.sched_getaffinity(0)), "kind": "oracle",
           "sample": "%d of %d streams of 1 of %d layers%s, %d decode steps (append + attention), median, "
                     "scaled linearly to all streams and layers" % (S, n_streams, n_layers,
                                                                     " at 1/%d of the context" % ctx_scale if ctx_scale > 1 else "",
                                                                     len(times)),
           "seconds_per_stream_step": t_stream, "scale_to_whole_step": scale}
    if t_one is not None:
        res["value_1_thread"] = value(t_one)
        res["seconds_per_stream_step_1_thread"] = t_one
    return res


def run_reference(args, rank, world):
    if rank != 0:
        return None
    w = W.config(args.config)
    n_layers = args.layers or w.n_layers
    warm = max(args.warmup, 3)                      # the arm under test never warms up with fewer steps
    ctx_start = ingest_context(w.ctx, args.steps, warm) + warm
    t0 = time.perf_counter()
    base = cpu_baseline(w, n_layers, ctx_start, budget_s=0.0, steps=args.warmup + args.steps)
    ms = (time.perf_counter() - t0) * 1e3
    return {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup,
            # what was timed: one stream of one layer per step; `value` scales it to the whole step
            "ms_per_step": base["seconds_per_stream_step"] * 1e3,
            "ms_per_step_is": "one sampled stream-step (append + attention of 1 of %d streams of 1 of %d layers); "
                              "value = batch * context / (ms_per_step * scale_to_whole_step)" % (w.batch * w.n_kv_heads, n_layers),
            "scale_to_whole_step": base["scale_to_whole_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, n_layers, ctx_start, world),
            "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "threads_used", "cores_available", "kind", "sample",
                                                  "value_1_thread") if k in base},
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_ms_total": ms}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload: 0..4 (default 2: Llama-8B-like batched decode); 5 = RD-V2 operating point; "
                                                          "6 = the paper's Quest setting (64-token pages, 12.5 %% of the pages)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the brief runs of the other workloads")
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
