#!/usr/bin/env python
"""Benchmark of the offloaded-MoE decode step (one line of JSON on stdout, rank 0).

Default workload: the Qwen3-VL-30B-A3B-shaped configuration (48 MoE layers, hidden 2048,
128 routed experts of intermediate 768, top-8, bf16 weights in pinned host memory, 16 HBM slots
per layer, rank-16 adapters, budget from the profiled window, batch 1), synthetic weights and
Zipf(1.1) token ids. A step is one decode step: one hidden row through all layers (router,
adapter, budget selection, asynchronous prefetch, on-demand loads, slot-indexed expert FFN).

  value : decode tokens/s, hidden rows already in HBM, timed with CUDA events on the compute stream
  e2e   : the same through spm_decode_step_host (pinned host rows in, host rows out, every step)
  roofline : expert-FFN kernel, algorithmic weight bytes / mean device time of its launches (CUDA
             event pair per launch, the kernel timed by itself on a fully-resident context; the
             same pair inside the main arm and the in-kernel windows are given beside it),
             against the measured HBM copy bandwidth
  cpu_baseline : the CPU oracle timed on this machine's host cores on a bounded sample

`--impl reference` times the CPU oracle instead (rank 0 only).
Multi-GPU: one process per GPU (torchrun), independent decode streams per rank, no collective on
the data path; value = all ranks' tokens / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import copy
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import synth

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from one ncu capture of a reduced
# case of the same workload (4 layers; a launch reads the same expert blobs whatever the layer count): 75.53 MB read +
# 0.8 - 1.2 MB written for the GEMV kernel, 306.7 + 8.7 MB for one 32-expert wave of the grouped kernel.
NCU_DRAM_BYTES_PER_LAUNCH = {"qwen3": 76.6e6, "batched_wave": 315.4e6}
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


# ------------------------------------------------------------------ helpers
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return json.load(open(p)), "measured"
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def dist_setup(backend: str):
    rank, local, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local, world


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def aggregate(elapsed_ms: float, tokens: int, world: int, device="cpu"):
    """(max-over-ranks time in ms, tokens summed over ranks)."""
    if world == 1:
        return elapsed_ms, tokens
    import torch.distributed as dist
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


class ClockSampler:
    """Samples SM clocks / throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.idx)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def hidden_rows(cfg, steps, stream):
    tok = synth.zipf_tokens(cfg, steps=steps, stream=stream)
    H = synth.embedding_rows(cfg, tok.reshape(-1))
    return tok, H.view(steps, cfg.batch, cfg.hidden).contiguous()


def affordable_store_layers(cfg, world):
    """Layers of experts this rank can keep pinned: all of them when 60 % of the host's available memory,
    split over the ranks of the node, holds the store; otherwise fewer, and the layers repeat (the context
    is told so through host_store_layers; sizes, copies and kernels are unchanged)."""
    per_layer = cfg.n_experts * cfg.expert_bytes
    try:
        avail = int(open("/proc/meminfo").read().split("MemAvailable:")[1].split()[0]) * 1024
    except Exception:
        return cfg.n_layers
    ranks = int(os.environ.get("LOCAL_WORLD_SIZE", world))
    return int(max(1, min(cfg.n_layers, (0.6 * avail / max(ranks, 1)) // per_layer)))


def workload_name(cfg):
    return (f"{cfg.name}: L{cfg.n_layers} D{cfg.hidden} n{cfg.n_experts} I{cfg.inter} K{cfg.top_k}"
            f"+{cfg.n_shared}sh r{cfg.adapter_rank} {cfg.dtype} slots{cfg.slots} batch{cfg.batch}")


def config_block(cfg, args):
    """What is run, in words both arms share (measured quantities live under `profile`)."""
    return {"workload": workload_name(cfg), "policy": "adapter",
            "budget_rule": "max(1, floor(window / t_xfer)) from the profiled window" if cfg.budget < 0 else f"fixed {cfg.budget}",
            "attention_stub_us": args.stub_us, "copy_delay_us": args.copy_delay_us, "seed": cfg.seed, "token_ids": "Zipf(1.1)",
            "l2": "inputs larger than L2: every layer streams its own slot pool, 3.6 GB of weights per step"}


def ffn_kernel_name(cfg):
    if cfg.batch > 1 and cfg.n_shared == 0 and cfg.dtype in ("bf16", "q4"):
        return "ffn_grouped_q4_kernel" if cfg.dtype == "q4" else "ffn_grouped_kernel"
    if cfg.dtype == "q4":
        return "ffn_gemv_q4_kernel"
    return "ffn_gemv_kernel"


def bench_config(args):
    """The named configuration; --layers / --slots shrink it for profiler captures and say so in its name."""
    cfg = synth.get_config(args.config)
    over = {}
    if args.layers:
        over["n_layers"] = args.layers
    if args.slots:
        over["slots"] = args.slots
    if over:
        cfg = cfg.replace(name=cfg.name + "-reduced", **over)
    return cfg


# ------------------------------------------------------------------ GPU arm
def timed_run(m, H_dev, first, count, world):
    """`count` decode steps starting at row `first`, device-timed on the compute stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out = torch.empty_like(H_dev[0])
    m.synchronize()
    barrier(world)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record(m.compute)
    for s in range(first, first + count):
        m.decode_step(H_dev[s], out)
    e1.record(m.compute)
    m.synchronize()
    torch.cuda.synchronize()
    wall = (time.perf_counter() - t0) * 1e3
    barrier(world)
    return e0.elapsed_time(e1), wall, out


def arm_summary(m, cfg, elapsed_ms, steps):
    st = m.stats()
    stall, ffn, n = m.layer_times()
    per = max(n, 1) * cfg.n_layers
    return {
        "tok_s": steps * cfg.batch / (elapsed_ms / 1e3),
        "stall_us_per_layer": float(stall.sum() / per),
        "router_done_to_ffn_done_us_per_layer": float((stall.sum() + ffn.sum()) / per),
        "ffn_us_per_launch": st["ffn_us"] / max(st["ffn_launches"], 1),
        "hit_rate": st["hits"] / max(st["hits"] + st["misses"], 1),
        "ready_recall": st["ready_sum"] / max(st["ready_count"], 1),
        "expert_recall_at_budget": (st["recall_sum"] / st["recall_count"]) if st["recall_count"] else None,
        "expert_recall_at_half_k_k_k_plus_2": [r / st["recall_count"] for r in st["recall_at"]] if st["recall_count"] else None,
        "copies_per_token": (st["misses"] + st["prefetch_issued"]) / max(steps * cfg.batch, 1),
        "prefetch_issued": st["prefetch_issued"], "prefetch_used": st["hits_prefetched"], "prefetch_wasted": st["wasted"],
        "late_arrivals": st["late_arrivals"],
        "h2d_gb_s_avg": st["h2d_bytes"] / (elapsed_ms / 1e3) / 1e9,
    }


def run_ours(args):
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.synth_model import build_from_synth
    from paper_2607_24787_b200.model import PinnedStore

    rank, local, world = dist_setup("nccl")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if rank == 0:
        build()
    barrier(world)
    cfg = bench_config(args)
    K, W = args.steps, args.warmup
    t_setup = time.time()
    store_layers = affordable_store_layers(cfg, world)
    m = build_from_synth(cfg, device=device, store_layers=store_layers)   # budget -1: profiled inside spm_init
    setup_s = time.time() - t_setup
    if args.stub_us:
        m.set_attention_stub_us(args.stub_us)
    if args.copy_delay_us:
        m.set_copy_delay_us(args.copy_delay_us)
    window_us, t_xfer_us, raw_budget = m.profile_window()
    budget = max(1, raw_budget) if cfg.budget < 0 else cfg.budget
    m.set_budget(budget)
    tok, H = hidden_rows(cfg, W + K, stream=rank)
    H_dev = H.to(device)
    H_pin = H.pin_memory()
    torch.cuda.synchronize()
    algo_bytes = (cfg.top_k + cfg.n_shared) * cfg.expert_bytes     # expert weight bytes per FFN launch

    # ---- main arm: adapter-guided prefetch, device-resident inputs ----------
    m.set_policy("adapter")
    m.set_timing(1)
    m.cache_reset()
    timed_run(m, H_dev, 0, W, world)
    m.reset_stats()
    clocks = ClockSampler(local)
    clocks.start()
    el_ms, wall_ms, _ = timed_run(m, H_dev, W, K, world)
    clk = clocks.stop()
    main = arm_summary(m, cfg, el_ms, K)
    st = m.stats()
    launches = st["kernel_launches"]
    ffn_us = st["ffn_us"] / max(st["ffn_launches"], 1)
    hint_events = m.events()
    el_max, tokens = aggregate(el_ms, K * cfg.batch, world, device)

    # ---- end to end: host rows in and out every step ------------------------
    m.cache_reset()
    out_pin = torch.empty(cfg.batch, cfg.hidden).pin_memory()
    for s in range(W):
        m.decode_step_host(H_pin[s], out_pin)
    barrier(world)
    t0 = time.perf_counter()
    for s in range(W, W + K):
        m.decode_step_host(H_pin[s], out_pin)
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_max, _ = aggregate(e2e_ms, K * cfg.batch, world, device)

    result = {
        "metric": "decode tokens/s with offloaded experts",
        "value": tokens / (el_max / 1e3), "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": el_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights, fp32 accumulate" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": config_block(cfg, args),
        "profile": {"budget": budget, "budget_raw": raw_budget, "window_us": window_us, "t_xfer_us": t_xfer_us,
                    "host_store_layers": store_layers, "setup_s": setup_s, "wall_ms_per_step": wall_ms / K},
        "clocks": clk,
        "e2e": {"value": tokens / (e2e_max / 1e3), "unit": "tokens/s",
                "h2d_bytes_per_step": cfg.batch * cfg.hidden * 4 + int(st["h2d_bytes"] / K),
                "d2h_bytes_per_step": cfg.batch * cfg.hidden * 4,
                "note": "h2d counts the hidden rows plus the mean expert bytes moved per step"},
        "gpu_launches": int(launches),
    }
    peaks, which = measured_peaks()
    peak = float(peaks.get("hbm_gbs", FALLBACK_HBM_GBS))
    achieved = algo_bytes / (ffn_us * 1e-6) / 1e9 if ffn_us > 0 else 0.0
    window_us = st["ffn_window_us"] / max(st["ffn_launches"], 1)
    # expert-FFN kernel inside the timed region of the main arm: CUDA event pair per launch.
    # Every launch here overlaps an in-flight prefetch copy, which by itself doubles the
    # duration of an HBM-streaming kernel on this machine; `isolated` (below, when the
    # resident leg runs) times the same entry point with no PCIe traffic.
    result["roofline"] = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                          "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(cfg.name), "kernel": ffn_kernel_name(cfg),
                          "peak_source": f"of {which}", "algorithmic_bytes_per_launch": algo_bytes,
                          "us_per_launch": ffn_us, "in_kernel_window_us": window_us,
                          "achieved_in_kernel_window": algo_bytes / (window_us * 1e-6) / 1e9 if window_us > 0 else None,
                          "frac_in_kernel_window": algo_bytes / (window_us * 1e-6) / 1e9 / peak if window_us > 0 else None,
                          "region": f"main arm, {K} timed steps x {cfg.n_layers} launches, each concurrent with a prefetch copy",
                          "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}
    result["main_arm"] = main

    if world == 1 and not args.no_arms:
        arms = {}
        n_arm = min(K, args.arm_steps)
        # on-demand loading (no prediction, no prefetch)
        m.set_policy("on_demand"); m.cache_reset()
        timed_run(m, H_dev, 0, W, world); m.reset_stats()
        el, _, _ = timed_run(m, H_dev, W, n_arm, world)
        arms["on_demand"] = arm_summary(m, cfg, el, n_arm)
        # perfect knowledge: the experts each layer truly needs, from the recorded routing of the main arm
        hint = [[[] for _ in range(cfg.n_layers)] for _ in range(W + K)]
        m.cache_reset(); m.set_policy("on_demand")
        timed_run(m, H_dev, 0, W + n_arm, world)
        for (s, l, kind, e, _) in m.events():
            if kind in ("HIT", "HIT_PREFETCHED", "MISS"):
                hint[s][l].append(e)
        m.set_policy("hint_trace"); m.set_hint_trace(hint); m.cache_reset()
        timed_run(m, H_dev, 0, W, world); m.reset_stats()
        el, _, _ = timed_run(m, H_dev, W, n_arm, world)
        arms["perfect_knowledge"] = arm_summary(m, cfg, el, n_arm)
        # on-demand and perfect knowledge again, with the FFN waiting for its copies on the device
        if cfg.batch == 1:
            m.set_device_wait(1)
            m.set_policy("on_demand"); m.cache_reset()
            timed_run(m, H_dev, 0, W, world); m.reset_stats()
            el, _, _ = timed_run(m, H_dev, W, n_arm, world)
            arms["on_demand_device_wait"] = arm_summary(m, cfg, el, n_arm)
            m.set_policy("hint_trace"); m.set_hint_trace(hint); m.cache_reset()
            timed_run(m, H_dev, 0, W, world); m.reset_stats()
            el, _, _ = timed_run(m, H_dev, W, n_arm, world)
            arms["perfect_knowledge_device_wait"] = arm_summary(m, cfg, el, n_arm)
            m.set_device_wait(0)
        # previous token's experts as the prediction (Naive Prefetch)
        m.set_policy("naive"); m.cache_reset()
        timed_run(m, H_dev, 0, W, world); m.reset_stats()
        el, _, _ = timed_run(m, H_dev, W, n_arm, world)
        arms["naive"] = arm_summary(m, cfg, el, n_arm)
        # prediction and control only (PRED0)
        m.set_policy("pred0"); m.cache_reset()
        timed_run(m, H_dev, 0, W, world); m.reset_stats()
        el, _, _ = timed_run(m, H_dev, W, n_arm, world)
        arms["pred0"] = arm_summary(m, cfg, el, n_arm)
        result["arms"] = arms
        # prefetch copy bandwidth: an uncontended batch of expert copies on the copy stream
        result["h2d"] = h2d_probe(m, cfg)

    if world == 1 and not args.no_resident:
        try:
            result["resident"] = resident_run(cfg, m, H_dev, W, min(K, args.arm_steps), peak, algo_bytes, device)
            b2b = result["resident"]["ffn_back_to_back"]
            iso = {
                "kernel": b2b["kernel"], "achieved": b2b["gb_s"], "frac": b2b["frac_of_measured_peak"],
                "us_per_launch": b2b["kernel_us"], "algorithmic_bytes_per_launch": b2b["algorithmic_bytes_per_launch"],
                "in_kernel_window_us": b2b["kernel_window_us"],
                "achieved_in_kernel_window": b2b["gb_s_in_kernel_window"],
                "frac_in_kernel_window": (b2b["gb_s_in_kernel_window"] or 0) / peak,
                "frac_of_nominal_8TBs": b2b["gb_s"] / NOMINAL_HBM_GBS,
                "region": (f"{b2b['launches']} launches of the kernel alone back to back on the compute stream (spm_time_ffn_kernel), "
                           "all experts resident, pools of all layers cycled (nothing served from L2), one CUDA event pair "
                           "around all of them, every launch with the programmatic-serialisation attribute all kernels of a decode step "
                           "carry: a launch requests its first weight rows while the FFN launch before it drains (inside a decode "
                           "step its predecessor is the routing kernel, so there us_per_launch_serialized applies); "
                           "us_per_launch = span / launches") if cfg.batch == 1 else
                          (f"{b2b['launches']} spm_moe_ffn launches back to back on the compute stream, all experts resident "
                           "(pools of all layers cycled, nothing served from L2), CUDA event pair per launch"),
                "us_per_launch_serialized": b2b.get("serialized_us"),
                "us_per_launch_graph_plain": b2b.get("graph_plain_us"),
                "frac_graph_plain": (b2b["algorithmic_bytes_per_launch"] / (b2b["graph_plain_us"] * 1e-6) / 1e9 / peak) if b2b.get("graph_plain_us") else None,
                "us_per_launch_graph_chained": b2b.get("graph_chained_us"),
                "frac_serialized": (b2b["algorithmic_bytes_per_launch"] / (b2b["serialized_us"] * 1e-6) / 1e9 / peak) if b2b.get("serialized_us") else None,
                "us_per_launch_event_pair_each": b2b["event_pair_each_us"],
                "frac_event_pair_each": b2b["algorithmic_bytes_per_launch"] / (b2b["event_pair_each_us"] * 1e-6) / 1e9 / peak}
            # The headline is the kernel timed by itself (burst peak as denominator). Inside the main arm every
            # launch follows a wait for PCIe copies and overlaps the next prefetch copy; an event pair there
            # measures mostly launch latency behind the busy link (the in-kernel window stays the same), so
            # that figure is kept beside it, not as the kernel's roofline.
            main_view = {k: result["roofline"][k] for k in ("achieved", "frac", "us_per_launch", "in_kernel_window_us",
                                                            "achieved_in_kernel_window", "frac_in_kernel_window", "region")}
            if cfg.batch > 1:      # a batched launch's bytes vary with the demand: only the isolated leg has a byte count
                main_view = {"us_per_launch": result["roofline"]["us_per_launch"], "region": result["roofline"]["region"]}
                result["roofline"]["traffic"] = None
            result["roofline"].update(iso)
            result["roofline"]["in_main_arm"] = main_view
        except Exception as e:   # noqa: BLE001 (reported, not hidden)
            result["resident"] = {"error": str(e)[:200]}

    if world == 1 and not args.no_arms and not args.no_extra and cfg.name == "qwen3":
        # what the targets are read from: exposed transfer time of the adapter-guided arm against on-demand loading
        # at the same slots, with the configuration's random adapters and with an informative stand-in (gate reuse)
        try:
            result["targets"] = targets_block(cfg, m, H_dev, W, min(K, args.arm_steps), result, device, hint)
        except Exception as e:   # noqa: BLE001
            result["targets"] = {"error": str(e)[:200]}
    if world == 1 and not args.no_extra and cfg.name == "qwen3":
        legs = {}
        for name, fn in (("batched", batched_leg), ("dsvl2", dsvl2_leg)):
            try:
                legs[name] = fn(args, m, peak, which, device)
            except Exception as e:   # noqa: BLE001 (reported, not hidden)
                legs[name] = {"error": str(e)[:300]}
        result["configs"] = legs

    # second denominator: what a kernel that only reads reaches on this device (the copy figure pays for writes too)
    try:
        ro = m.measure_read_bandwidth(4 << 30)
        result["roofline"]["read_only_stream_gb_s"] = ro
        result["roofline"]["frac_of_read_only_stream"] = result["roofline"]["achieved"] / ro
    except Exception as e:   # noqa: BLE001 (pools smaller than 256 MiB: nothing to measure)
        result["roofline"]["read_only_stream_gb_s"] = None
    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        try:
            result["cpu_baseline"] = cpu_baseline(args, cfg, budget)
        except Exception as e:   # noqa: BLE001 (reported, not hidden)
            result["cpu_baseline"] = {"error": str(e)[:300]}
    m.close()
    if rank == 0:
        print(json.dumps(result))


def run_arm(ctx, cfg, H_dev, W, n, policy, hint=None):
    ctx.set_policy(policy)
    if hint is not None:
        ctx.set_hint_trace(hint)
    ctx.set_timing(1); ctx.cache_reset()
    timed_run(ctx, H_dev, 0, W, 1); ctx.reset_stats()
    el, _, _ = timed_run(ctx, H_dev, W, n, 1)
    return arm_summary(ctx, cfg, el, n)


def paper_regime_block(cfg, m, g, H_dev, W, n, hint, t_xfer_us):
    """The same arms with an attention stand-in of two transfer times per layer in front of every router, which
    makes the overlap window about as wide as the paper's (two transfers, Figure 1b): the budget is then the
    profiled floor(window / t_xfer), and prefetching has something to hide behind."""
    stub = int(round(2 * t_xfer_us))
    keep = (m.get_budget(), g.get_budget())
    out = {"attention_stub_us": stub, "steps_per_arm": n}
    try:
        for ctx in (m, g):
            ctx.set_attention_stub_us(stub)
        window_us, t_us, raw = m.profile_window()
        budget = max(1, raw)
        out.update(window_us=window_us, t_xfer_us=t_us, budget_raw=raw, budget=budget)
        for ctx in (m, g):
            ctx.set_budget(budget)
        arms = {"on_demand": run_arm(m, cfg, H_dev, W, n, "on_demand"),
                "adapter_random": run_arm(m, cfg, H_dev, W, n, "adapter"),
                "adapter_gate_reuse": run_arm(g, cfg, H_dev, W, n, "adapter"),
                "perfect_knowledge": run_arm(m, cfg, H_dev, W, n, "hint_trace", hint)}
        od = arms["on_demand"]
        for k, a in arms.items():
            out[k] = {"tok_s": a["tok_s"], "stall_us_per_layer": a["stall_us_per_layer"], "ready_recall": a["ready_recall"],
                      "expert_recall_at_budget": a["expert_recall_at_budget"], "gain_over_on_demand": a["tok_s"] / od["tok_s"] - 1.0}
    finally:
        for ctx, b in zip((m, g), keep):
            ctx.set_attention_stub_us(0)
            ctx.set_budget(b)
    return out


def targets_block(cfg, m, H_dev, W, n_arm, result, device, hint=None):
    """Exposed (non-overlapped) transfer time per layer: adapter arms against on-demand loading, same slots."""
    from paper_2607_24787_b200.synth_model import build_from_synth
    od = result["arms"]["on_demand"]
    out = {"slots": cfg.slots, "steps_per_arm": n_arm,
           "on_demand": {"stall_us_per_layer": od["stall_us_per_layer"], "tok_s": od["tok_s"]},
           "adapter_random": {"stall_us_per_layer": result["main_arm"]["stall_us_per_layer"], "tok_s": result["main_arm"]["tok_s"],
                              "expert_recall_at_budget": result["main_arm"]["expert_recall_at_budget"]},
           "perfect_knowledge": {"stall_us_per_layer": result["arms"]["perfect_knowledge"]["stall_us_per_layer"],
                                 "tok_s": result["arms"]["perfect_knowledge"]["tok_s"]}}
    g = build_from_synth(cfg, budget=result["profile"]["budget"], device=device, store=m.store, adapter="gate_reuse",
                         store_layers=m.store_layers)
    g.set_policy("adapter"); g.set_timing(1); g.cache_reset()
    timed_run(g, H_dev, 0, W, 1); g.reset_stats()
    el, _, _ = timed_run(g, H_dev, W, n_arm, 1)
    a = arm_summary(g, cfg, el, n_arm)
    if hint is not None:
        try:
            out["paper_regime"] = paper_regime_block(cfg, m, g, H_dev, W, min(32, n_arm), hint, result["profile"]["t_xfer_us"])
        except Exception as e:   # noqa: BLE001 (reported, not hidden)
            out["paper_regime"] = {"error": str(e)[:200]}
    g.close()
    out["adapter_gate_reuse"] = {"stall_us_per_layer": a["stall_us_per_layer"], "tok_s": a["tok_s"],
                                 "expert_recall_at_budget": a["expert_recall_at_budget"], "ready_recall": a["ready_recall"]}
    out["exposed_below_on_demand"] = {k: out[k]["stall_us_per_layer"] < od["stall_us_per_layer"]
                                      for k in ("adapter_random", "adapter_gate_reuse", "perfect_knowledge")}
    return out


def leg_offloaded(m, cfg, H_dev, W, K):
    m.set_policy("adapter"); m.set_timing(1); m.cache_reset()
    timed_run(m, H_dev, 0, W, 1); m.reset_stats()
    el, _, _ = timed_run(m, H_dev, W, K, 1)
    out = arm_summary(m, cfg, el, K)
    st = m.stats()
    out["steps"] = K
    out["gpu_launches"] = int(st["kernel_launches"])
    return out, st


def batched_leg(args, m, peak, which, device):
    """Batched decode on the Qwen3 shape (64 sequences, 32 slots per layer), on the pinned store the main arm
    filled: offloaded tokens/s, then the grouped tcgen05 kernel by itself at the size of one wave (the 32 experts a
    pool holds: 302 MB) and with every expert resident (about 120 distinct experts per launch: 1.1 GB)."""
    from paper_2607_24787_b200.synth_model import build_from_synth
    cfg = synth.get_config("batched")
    W, K = 3, max(2, min(args.steps, args.batched_steps))
    mb = build_from_synth(cfg, device=device, store=m.store, store_layers=m.store_layers)     # budget -1: profiled
    window_us, t_xfer_us, raw = mb.get_profile()
    _, H = hidden_rows(cfg, W + K, stream=0)
    H_dev = H.to(device)
    torch.cuda.synchronize()
    out = {"workload": workload_name(cfg), "profile": {"window_us": window_us, "t_xfer_us": t_xfer_us, "budget_raw": raw,
                                                        "budget": mb.get_budget()}}
    off, st = leg_offloaded(mb, cfg, H_dev, W, K)
    out["offloaded"] = off
    if st["ffn_us"] > 0:
        # inside the offloaded run every launch is one wave; its bytes are the experts that wave computes
        wave_bytes = (st["hits"] + st["misses"]) * cfg.expert_bytes / max(st["ffn_launches"], 1)
        us = st["ffn_us"] / max(st["ffn_launches"], 1)
        out["offloaded"]["ffn_wave_in_run"] = {"us_per_launch": us, "algorithmic_bytes_per_launch": wave_bytes,
                                                "gb_s": wave_bytes / (us * 1e-6) / 1e9, "launches": int(st["ffn_launches"])}
    # the same steps with the grouped kernel's producer warp waiting for the copies itself (per unit) instead of the
    # host ordering each launch behind the copy events
    try:
        mb.set_device_wait(1)
        dw, _ = leg_offloaded(mb, cfg, H_dev, W, K)
        out["offloaded_device_wait"] = {k: dw[k] for k in ("tok_s", "stall_us_per_layer", "router_done_to_ffn_done_us_per_layer",
                                                          "late_arrivals", "h2d_gb_s_avg")}
    except Exception as e:   # noqa: BLE001 (no stream-ordered memory writes on this driver)
        out["offloaded_device_wait"] = {"error": str(e)[:200]}
    mb.set_device_wait(0)
    # one wave by itself: the first `slots` experts of every layer resident, tokens routed among them (all hits)
    mb.cache_reset(); mb.set_policy("on_demand")
    S = cfg.slots
    for l in range(cfg.n_layers):
        mb.prefetch_async(l, np.arange(S, dtype=np.int32))
    mb.synchronize()
    out["roofline_wave"] = grouped_alone(cfg, mb, S, peak, which, launches=96)
    mb.close()
    full = build_from_synth(cfg, slots=cfg.n_experts, budget=0, device=device, store=m.store, store_layers=m.store_layers)
    full.set_policy("on_demand")
    for l in range(cfg.n_layers):
        full.prefetch_async(l, np.arange(cfg.n_experts, dtype=np.int32))
    full.synchronize()
    out["roofline"] = grouped_alone(cfg, full, cfg.n_experts, peak, which, launches=96)
    full.set_timing(0)
    for _ in range(3):
        timed_run(full, H_dev, 0, W, 1)
    el, _, _ = timed_run(full, H_dev, W, K, 1)
    out["resident_host_free_tok_s"] = K * cfg.batch / (el / 1e3)
    full.close()
    return out


def grouped_alone(cfg, ctx, n_resident, peak, which, launches):
    """`launches` spm_moe_ffn calls back to back, every token's K experts drawn among the first `n_resident`
    (all resident): CUDA event pair around each grouped-kernel launch (gather and combine kernels outside it)."""
    rng = np.random.default_rng(1)
    nb = cfg.batch
    x = torch.randn(nb, cfg.hidden, device=ctx.device)
    w = torch.full((nb, cfg.top_k), 1.0 / cfg.top_k, device=ctx.device)
    h = torch.zeros(nb, cfg.hidden, device=ctx.device)
    ids = [np.stack([np.sort(rng.permutation(n_resident)[:cfg.top_k]) for _ in range(nb)]).astype(np.int32) for _ in range(launches)]
    mean_bytes = float(np.mean([len(np.unique(i)) * cfg.expert_bytes for i in ids]))
    torch.cuda.synchronize()
    ctx.set_timing(1)
    for i in range(8):
        ctx.moe_ffn(i % cfg.n_layers, x, ids[i], w, h)
    ctx.reset_stats()
    for i in range(launches):
        ctx.moe_ffn(i % cfg.n_layers, x, ids[i], w, h)
    ctx.synchronize()
    st = ctx.stats()
    us = st["ffn_us"] / max(st["ffn_launches"], 1)
    ach = mean_bytes / (us * 1e-6) / 1e9
    win = st["ffn_window_us"] / max(st["ffn_launches"], 1)      # in-kernel clock: first CTA past its dependency wait -> last CTA end
    return {"bound": "hbm", "kernel": ffn_kernel_name(cfg), "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
            "in_kernel_window_us": win, "frac_in_kernel_window": mean_bytes / (win * 1e-6) / 1e9 / peak if win > 0 else None,
            "traffic": NCU_DRAM_BYTES_PER_LAUNCH["batched_wave"] if (cfg.name == "batched" and n_resident == cfg.slots) else None,
            "peak_source": f"of {which}", "algorithmic_bytes_per_launch": mean_bytes, "us_per_launch": us,
            "launches": int(st["ffn_launches"]), "misses": int(st["misses"]), "distinct_experts_per_launch": mean_bytes / cfg.expert_bytes,
            "region": f"{launches} spm_moe_ffn launches back to back, {nb} tokens x top-{cfg.top_k} among {n_resident} resident "
                      "experts per layer, pools of all layers cycled, CUDA event pair per grouped-kernel launch"}


def dsvl2_leg(args, m, peak, which, device):
    """DeepSeek-VL2-Tiny-shaped decode (12 layers, hidden 1280, 64 experts of intermediate 896, top-6 + 2 shared,
    8 slots): offloaded tokens/s with its own 5.3 GB pinned store, and the GEMV expert kernel by itself."""
    from paper_2607_24787_b200.synth_model import build_from_synth
    cfg = synth.get_config("dsvl2")
    W, K = 3, max(2, min(args.steps, args.dsvl2_steps))
    md = build_from_synth(cfg, device=device)
    window_us, t_xfer_us, raw = md.get_profile()
    _, H = hidden_rows(cfg, W + K, stream=0)
    H_dev = H.to(device)
    torch.cuda.synchronize()
    out = {"workload": workload_name(cfg), "profile": {"window_us": window_us, "t_xfer_us": t_xfer_us, "budget_raw": raw,
                                                        "budget": md.get_budget()}}
    out["offloaded"], _ = leg_offloaded(md, cfg, H_dev, W, K)
    md.set_policy("on_demand"); md.cache_reset()
    timed_run(md, H_dev, 0, W, 1); md.reset_stats()
    el, _, _ = timed_run(md, H_dev, W, K, 1)
    od = arm_summary(md, cfg, el, K)
    out["on_demand"] = {"tok_s": od["tok_s"], "stall_us_per_layer": od["stall_us_per_layer"]}
    full = build_from_synth(cfg, slots=cfg.n_experts, budget=0, device=device, store=md.store)
    full.set_policy("on_demand")
    for l in range(cfg.n_layers):
        full.prefetch_async(l, np.arange(cfg.n_experts, dtype=np.int32))
    full.synchronize()
    algo = (cfg.top_k + cfg.n_shared) * cfg.expert_bytes
    b2b = ffn_back_to_back(cfg, full, algo, peak, launches=240)
    out["roofline"] = {"bound": "hbm", "kernel": b2b["kernel"], "achieved": b2b["gb_s"], "peak": peak, "unit": "GB/s",
                       "frac": b2b["frac_of_measured_peak"], "traffic": None, "peak_source": f"of {which}",
                       "algorithmic_bytes_per_launch": algo, "us_per_launch": b2b["kernel_us"],
                       "us_per_launch_serialized": b2b.get("serialized_us"),
                       "frac_serialized": (algo / (b2b["serialized_us"] * 1e-6) / 1e9 / peak) if b2b.get("serialized_us") else None,
                       "us_per_launch_graph_plain": b2b.get("graph_plain_us"),
                       "frac_graph_plain": (algo / (b2b["graph_plain_us"] * 1e-6) / 1e9 / peak) if b2b.get("graph_plain_us") else None,
                       "us_per_launch_graph_chained": b2b.get("graph_chained_us"),
                       "us_per_launch_event_pair_each": b2b["event_pair_each_us"],
                       "in_kernel_window_us": b2b.get("chained_window_us"),
                       "region": "240 launches of the kernel alone back to back (spm_time_ffn_kernel, programmatic dependent "
                                 "launch), all experts resident, one CUDA event pair around all of them"}
    full.set_timing(0)
    for _ in range(3):
        timed_run(full, H_dev, 0, W, 1)
    el, _, _ = timed_run(full, H_dev, W, K, 1)
    out["resident_host_free_tok_s"] = K * cfg.batch / (el / 1e3)
    full.close()
    md.close()
    return out


def h2d_probe(m, cfg):
    """Mean bandwidth of 8 back-to-back expert copies pinned host -> HBM, against one large copy."""
    n = 8
    blob = cfg.expert_bytes
    dst = torch.empty(n * blob, dtype=torch.uint8, device=m.device)
    src = m.store.tensor
    big = min(src.numel(), 1 << 30)
    dst_big = torch.empty(big, dtype=torch.uint8, device=m.device)
    s = m.copy
    best_small, best_big = 0.0, 0.0
    with torch.cuda.stream(s):
        for it in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s)
            for i in range(n):
                off = ((it * n + i) * 17 % (cfg.n_layers * cfg.n_experts)) * blob
                dst[i * blob:(i + 1) * blob].copy_(src[off:off + blob], non_blocking=True)
            e1.record(s); e1.synchronize()
            best_small = max(best_small, n * blob / (e0.elapsed_time(e1) * 1e-3) / 1e9)
            e0.record(s)
            dst_big.copy_(src[:big], non_blocking=True)
            e1.record(s); e1.synchronize()
            best_big = max(best_big, big / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    return {"expert_copies_gb_s": best_small, "pinned_peak_gb_s": best_big, "frac": best_small / best_big,
            "copy_bytes": blob}


def resident_run(cfg, m, H_dev, W, K, peak, algo_bytes, device):
    """All experts resident (slots = n): the HBM-bound ceiling and the FFN kernel without PCIe traffic."""
    from paper_2607_24787_b200.synth_model import build_from_synth
    full = build_from_synth(cfg, slots=cfg.n_experts, budget=0, device=device, store=m.store, max_batch=cfg.batch,
                            store_layers=m.store_layers)
    full.set_policy("on_demand")
    for l in range(cfg.n_layers):                          # preload every expert
        full.prefetch_async(l, np.arange(cfg.n_experts, dtype=np.int32))
    full.synchronize()
    full.set_timing(1)
    # host-driven leg: one host turn per layer, an event pair around every FFN kernel
    full.set_host_free(0)
    timed_run(full, H_dev, 0, W, 1)
    full.reset_stats()
    el, _, _ = timed_run(full, H_dev, W, K, 1)
    st = full.stats()
    stall, ffn, n = full.layer_times()
    ffn_us = st["ffn_us"] / max(st["ffn_launches"], 1)
    ach = algo_bytes / (ffn_us * 1e-6) / 1e9
    out = {"tok_s": K * cfg.batch / (el / 1e3), "misses": st["misses"], "ffn_us_per_launch": ffn_us,
           "stall_us_per_layer": float(stall.sum() / (max(n, 1) * cfg.n_layers))}
    if cfg.batch == 1:
        out.update(ffn_gb_s=ach, ffn_frac_of_measured_peak=ach / peak)
    # host-free leg: all layers enqueued without waiting for routing results, kernels launched
    # ahead of their predecessor's end (no per-kernel events: the in-kernel window is reported)
    full.set_host_free(1)
    for policy in ("on_demand", "adapter"):
        full.set_policy(policy)
        timed_run(full, H_dev, 0, W, 1)
        full.reset_stats()
        el, _, _ = timed_run(full, H_dev, W, K, 1)
        st = full.stats()
        nl = max(st["ffn_launches"], 1)
        leg = {"tok_s": K * cfg.batch / (el / 1e3), "us_per_layer": el * 1e3 / (K * cfg.n_layers),
               "host_free_steps": st["host_free_steps"], "misses": st["misses"],
               "router_window_us": st["router_window_us"] / nl, "reduce_window_us": st["reduce_window_us"] / nl,
               "idle_between_kernels_us_per_layer": st["gap_us"] / nl}
        if st["host_free_steps"] and st["ffn_window_us"] > 0:
            win = st["ffn_window_us"] / max(st["ffn_launches"], 1)
            leg.update(ffn_window_us=win, ffn_gb_s_in_window=algo_bytes / (win * 1e-6) / 1e9,
                       ffn_frac_in_window=algo_bytes / (win * 1e-6) / 1e9 / peak,
                       hbm_bound_tok_s=peak * 1e9 / (algo_bytes * cfg.n_layers) * cfg.batch)
        # the same without per-kernel clocks, launch by launch and replayed from CUDA graphs
        full.set_timing(0)
        for replay, key in ((0, "tok_s_untimed_launches"), (1, "tok_s_untimed_graph_replay")):
            full.set_graph_replay(replay)
            for _ in range(1 + 9 // max(W, 1)):       # one step launch by launch, then one capture per trace slot (8)
                timed_run(full, H_dev, 0, W, 1)
            el2, _, _ = timed_run(full, H_dev, W, K, 1)
            leg[key] = K * cfg.batch / (el2 / 1e3)
        full.set_graph_replay(1)
        full.set_timing(1)
        out["host_free_" + policy] = leg
    full.set_policy("on_demand")
    full.set_host_free(0)
    out["ffn_back_to_back"] = ffn_back_to_back(cfg, full, algo_bytes, peak)
    full.close()
    return out


def ffn_back_to_back(cfg, full, algo_bytes, peak, launches=480):
    """The expert-FFN entry point alone: `launches` spm_moe_ffn calls enqueued back to back on a
    fully-resident context, cycling through all layers' pools (54 GiB, so nothing is served from L2),
    each launch bracketed by a CUDA event pair on the compute stream, plus one pair around them all.
    With several sequences per step every token draws K distinct experts at random, so a launch
    streams (number of distinct experts) blobs through the grouped tensor-core kernel."""
    rng = np.random.default_rng(0)
    nb = cfg.batch
    if nb > 1:
        launches = min(launches, 96)
    x = torch.randn(nb, cfg.hidden, device=full.device)
    w = torch.full((nb, cfg.top_k), 1.0 / cfg.top_k, device=full.device)
    h = torch.zeros(nb, cfg.hidden, device=full.device)
    ids = [np.stack([np.sort(rng.permutation(cfg.n_experts)[:cfg.top_k]) for _ in range(nb)]).astype(np.int32)
           for _ in range(launches)]
    per_launch_bytes = [(len(np.unique(i)) + cfg.n_shared) * cfg.expert_bytes for i in ids]
    mean_bytes = float(np.mean(per_launch_bytes))
    torch.cuda.synchronize()
    full.set_timing(1)
    for i in range(16):
        full.moe_ffn(i % cfg.n_layers, x, ids[i], w, h)
    full.reset_stats()
    for i in range(launches):
        full.moe_ffn(i % cfg.n_layers, x, ids[i], w, h)
    full.synchronize()
    st = full.stats()
    per_kernel = st["ffn_us"] / max(st["ffn_launches"], 1)
    window = st["ffn_window_us"] / max(st["ffn_launches"], 1)
    # the same calls without per-launch events: one pair around all of them (kernel + combine + gaps)
    full.set_timing(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(full.compute)
    for i in range(launches):
        full.moe_ffn(i % cfg.n_layers, x, ids[i], w, h)
    e1.record(full.compute)
    full.synchronize()
    per_call = e0.elapsed_time(e1) * 1e3 / launches
    out = {"launches": launches, "kernel": ffn_kernel_name(cfg),
           "algorithmic_bytes_per_launch": mean_bytes, "event_pair_each_us": per_kernel,
           "kernel_window_us": window if window > 0 else None, "call_us_incl_combine": per_call,
           "misses": st["misses"]}
    if nb == 1:
        # the kernel alone, no combine in between: one event pair around all launches. `chained`: launched as a
        # decode step launches it (programmatic dependent launch: a launch fetches its first weight rows while its
        # predecessor drains); `serialized`: plain launches, each starts after the one before it has ended.
        ids1 = np.stack([i[0] for i in ids]).astype(np.int32)
        full.time_ffn_kernel(0, x[0], ids1[:32], w[0], chained=True)          # warm-up
        chained = [full.time_ffn_kernel(0, x[0], ids1, w[0], chained=True) for _ in range(3)]
        serial = [full.time_ffn_kernel(0, x[0], ids1, w[0], chained=False) for _ in range(3)]
        out["chained_us"] = statistics.median(c[0] for c in chained)
        out["chained_window_us"] = statistics.median(c[1] for c in chained)
        out["serialized_us"] = statistics.median(c[0] for c in serial)
        out["serialized_window_us"] = statistics.median(c[1] for c in serial)
        # the same two launch sequences captured into one CUDA graph and replayed (how a host-free decode step is launched)
        try:
            out["graph_plain_us"] = statistics.median(full.time_ffn_kernel(0, x[0], ids1, w[0], chained=2)[0] for _ in range(3))
            out["graph_chained_us"] = statistics.median(full.time_ffn_kernel(0, x[0], ids1, w[0], chained=3)[0] for _ in range(3))
        except Exception as e:   # noqa: BLE001 (reported, not hidden)
            out["graph_error"] = str(e)[:200]
        per_kernel = out["chained_us"]
    out["kernel_us"] = per_kernel
    ach = mean_bytes / (per_kernel * 1e-6) / 1e9
    out.update(gb_s=ach, frac_of_measured_peak=ach / peak,
               gb_s_in_kernel_window=mean_bytes / (window * 1e-6) / 1e9 if window > 0 else None)
    return out


def run_sweep(args):
    """Budget x cache-size sweep on the Qwen3-shaped model: for every slots-per-layer value the
    on-demand arm, and per budget the adapter arm (the configuration's random adapters), adapter
    arms with structured stand-ins for trained weights (gate reuse, truncated SVD of the next
    gate, reduced-rank regression on a calibration stream) and the perfect-knowledge arm."""
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.synth_model import build_from_synth, collect_router_io, fitted_adapters
    build()
    device = "cuda:0"
    torch.cuda.set_device(0)
    cfg = bench_config(args)
    K, W = args.steps, args.warmup
    tok, H = hidden_rows(cfg, W + K, stream=0)
    H_dev = H.to(device)
    torch.cuda.synchronize()
    store, cells = None, []
    budgets = [int(b) for b in args.sweep_budgets.split(",")]
    kinds = args.sweep_adapters.split(",")
    if "random" not in kinds:
        kinds.insert(0, "random")            # the on-demand and perfect-knowledge arms ride on this context
    kinds.sort(key=lambda k: k != "random")
    fitted = None
    for S in [int(x) for x in args.sweep_slots.split(",")]:
        for kind in kinds:
            adapter = fitted if kind == "fit" else kind
            m = build_from_synth(cfg, slots=S, budget=1, device=device, store=store, adapter=adapter)
            store = m.store
            m.set_timing(1)
            if args.stub_us:
                m.set_attention_stub_us(args.stub_us)
            if args.copy_delay_us:
                m.set_copy_delay_us(args.copy_delay_us)
            if kind == "random":
                window = m.profile_window()
                if "fit" in kinds and fitted is None:
                    # calibration stream independent of the evaluated one (its own generator stream)
                    _, Hc = hidden_rows(cfg, args.calib_steps, stream=777)
                    X, Z = collect_router_io(m, Hc.to(device))
                    fitted = fitted_adapters(X, Z, cfg.adapter_rank, cfg.torch_dtype)
                    del X, Z

            def arm(policy, budget, hint=None):
                m.set_policy(policy); m.set_budget(budget)
                if hint is not None:
                    m.set_hint_trace(hint)
                m.cache_reset()
                timed_run(m, H_dev, 0, W, 1); m.reset_stats()
                el, _, _ = timed_run(m, H_dev, W, K, 1)
                out = arm_summary(m, cfg, el, K)
                out.update(slots=S, budget=budget, policy=policy if kind == "random" or policy != "adapter" else "adapter_" + kind)
                return out

            if kind == "random":
                cells.append(arm("on_demand", 0))
                hint = [[[] for _ in range(cfg.n_layers)] for _ in range(W + K)]
                m.set_policy("on_demand"); m.cache_reset()
                timed_run(m, H_dev, 0, W + K, 1)
                for (s_, l_, kind_, e_, _) in m.events():
                    if kind_ in ("HIT", "HIT_PREFETCHED", "MISS"):
                        hint[s_][l_].append(e_)
                for b in budgets:
                    cells.append(arm("adapter", b))
                    cells.append(arm("hint_trace", b, hint))
            else:
                for b in budgets:
                    cells.append(arm("adapter", b))
            m.close()
    print(json.dumps({"sweep": f"{cfg.name}: {K} steps per cell, seed {cfg.seed}", "attention_stub_us": args.stub_us,
                      "window_us": window[0], "t_xfer_us": window[1], "budget_raw": window[2], "cells": cells}))


# ------------------------------------------------------------------ CPU oracle legs
class LazyWeights:
    """Oracle weight provider: matrices regenerated from the synthetic generator on first use."""

    def __init__(self, cfg, device):
        self.cfg, self.dev, self.cache = cfg, device, {}

    def _get(self, key, fn):
        if key not in self.cache:
            self.cache[key] = fn()
        return self.cache[key]

    @staticmethod
    def _f64(t):
        return t.to("cpu").to(torch.float64).numpy()

    def gamma(self, l):
        return np.ones(self.cfg.hidden)

    def router(self, l):
        return self._get(("r", l), lambda: self._f64(synth.router_w(self.cfg, l, self.dev)))

    def adapter(self, l):
        return self._get(("a", l), lambda: (self._f64(synth.adapter_a(self.cfg, l, self.dev)),
                                            self._f64(synth.adapter_b(self.cfg, l, self.dev))))

    def expert(self, l, e):
        def gen():
            g, u, d = synth.expert_matrices(self.cfg, l, [e], self.dev)
            return self._f64(g[0]), self._f64(u[0]), self._f64(d[0])
        return self._get(("e", l, e), gen)

    def shared(self, l):
        return [self.expert(l, self.cfg.n_experts + s) for s in range(self.cfg.n_shared)]


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


class blas_threads:
    """Pins the thread count of every BLAS / OpenMP pool numpy and torch use, for the duration of a block."""

    def __init__(self, n):
        self.n, self.ctx, self.torch_before = n, None, None

    def __enter__(self):
        try:
            from threadpoolctl import threadpool_limits
            self.ctx = threadpool_limits(limits=self.n)
            self.ctx.__enter__()
        except Exception:
            self.ctx = None
        self.torch_before = torch.get_num_threads()
        torch.set_num_threads(self.n)
        return self

    def __exit__(self, *exc):
        torch.set_num_threads(self.torch_before)
        if self.ctx is not None:
            self.ctx.__exit__(*exc)


def make_oracle(cfg, wts, budget, slots=None, policy="adapter"):
    from oracle.ref_decode import RefDecoder
    return RefDecoder(cfg.n_layers, cfg.hidden, cfg.n_experts, cfg.top_k, wts, cfg.slots if slots is None else slots,
                      budget, policy=policy, renormalize=bool(cfg.renormalize), rms_eps=cfg.rms_eps, keep_records=False)


def oracle_steps(cfg, H, device, budget, threads, layers=None, mem_budget=40e9):
    """Times the oracle, as it stands, on the decode steps H[s] with `threads` BLAS threads.
    Weights are generated before the clock starts: an untimed pass of the same step from a copy of
    the decoder's cache state asks the provider for exactly the experts the timed step will ask for
    (demanded and prefetched), and the provider's cache is emptied after the step. The fp64 matrices of one step stay below
    `mem_budget` bytes: a batched step touches nearly every expert of every layer, so there the
    sample is the first Ls layers. Returns (seconds per step, list; layers used)."""
    per_layer = min(cfg.n_experts, cfg.batch * cfg.top_k) * 3 * cfg.inter * cfg.hidden * 8
    Ls = int(max(1, min(cfg.n_layers, mem_budget // max(per_layer, 1))))
    if layers:
        Ls = min(Ls, layers)
    sub = cfg.replace(n_layers=Ls) if Ls < cfg.n_layers else cfg
    wts = LazyWeights(sub, device if torch.cuda.is_available() else "cpu")
    ref = make_oracle(sub, wts, budget)
    times = []
    with blas_threads(threads):
        for s in range(H.shape[0]):
            dry = copy.copy(ref)                 # same slot-table state, same weights: untimed, fills the weight cache for this step
            dry.table = copy.deepcopy(ref.table)
            dry.storage = [dict(d) for d in ref.storage]
            dry.prev_rank = [list(r) for r in ref.prev_rank]
            dry.step(H[s])
            del dry
            t0 = time.perf_counter()
            ref.step(H[s])
            times.append(time.perf_counter() - t0)
            wts.cache = {k: v for k, v in wts.cache.items() if k[0] != "e"}   # bound memory
    return times, Ls


ORACLE_THREADS = 1      # the headline reading: steady from step to step (with every core the same steps read 2.6 - 8.6 tokens/s within one run)


def cpu_baseline(args, cfg, budget):
    """The oracle on a bounded sample, timed in a process of its own: `bench.py --impl reference` on the first decode
    steps of the bench's token stream, on ORACLE_THREADS pinned thread(s) (the headline: reproducible), and once with
    every host core the process may use. A process of its own, so that the figure is the one the reference arm gives."""
    def run(steps, threads):
        cmd = [sys.executable, os.path.abspath(__file__), "--impl", "reference", "--config", args.config, "--steps", str(steps),
               "--warmup", "3", "--oracle-threads", str(threads), "--oracle-budget", str(budget)]
        if args.layers:
            cmd += ["--layers", str(args.layers)]
        if args.slots:
            cmd += ["--slots", str(args.slots)]
        env = dict(os.environ)
        for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
            env.pop(k, None)
        out = subprocess.run(cmd, capture_output=True, text=True, timeout=1200, env=env)
        lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
        if out.returncode != 0 or not lines:
            raise RuntimeError("reference arm failed: " + out.stderr[-300:])
        return json.loads(lines[-1])
    one = run(max(2, args.cpu_steps), ORACLE_THREADS)
    cores = host_cores()
    wide = run(2, cores)
    per_step = one["step_tok_s"]
    value = statistics.median(per_step)      # (the first timed step of a fresh process is the slow one)
    return {"value": value, "unit": "tokens/s", "cores": ORACLE_THREADS, "kind": "oracle",
            "per_step": per_step, "mean": one["value"], "spread": (max(per_step) - min(per_step)) / value,
            "all_host_cores": {"value": wide["value"], "cores": cores, "sample": wide["cpu_baseline"]["sample"]},
            "sample": one["cpu_baseline"]["sample"] + f"; median of {len(per_step)} steps after 3 warm-up steps, in a process of its own"}


def run_reference(args):
    rank, local, world = dist_env()
    if rank != 0:
        return
    cfg = bench_config(args)
    K, W = args.steps, args.warmup
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    # a step = one decode step over the first Ls layers, Ls sized so the run ends within minutes
    per_layer_s = 0.05
    Ls = int(max(1, min(cfg.n_layers, 150.0 / max((K + W) * per_layer_s * 2, 1e-9))))
    _, H = hidden_rows(cfg, W + K, stream=0)
    H = H.numpy()
    budget = args.oracle_budget if args.oracle_budget >= 0 else (1 if cfg.budget < 0 else cfg.budget)
    cores = args.oracle_threads if args.oracle_threads > 0 else ORACLE_THREADS
    times, Ls = oracle_steps(cfg, H, dev, budget, cores, layers=Ls)
    dt = sum(times[W:])
    tok_s = K * cfg.batch * (Ls / cfg.n_layers) / dt
    sample = (f"each step = one decode step over the first {Ls} of {cfg.n_layers} layers, numpy fp64 oracle, "
              f"weights pre-generated, BLAS pinned to {cores} thread(s); tokens/s scaled by {Ls}/{cfg.n_layers}")
    print(json.dumps({
        "impl": "reference", "metric": "decode tokens/s with offloaded experts", "value": tok_s, "unit": "tokens/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": dt / K * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_block(cfg, args),
        "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "step_tok_s": [cfg.batch * (Ls / cfg.n_layers) / t for t in times[W:]],
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="qwen3", choices=list(synth.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="reduced layer count (profiler captures only)")
    ap.add_argument("--slots", type=int, default=0, help="override slots per layer")
    ap.add_argument("--arm-steps", type=int, default=128)
    ap.add_argument("--cpu-steps", type=int, default=3)
    ap.add_argument("--sweep", action="store_true", help="budget x slots sweep (prints one JSON object with all cells)")
    ap.add_argument("--sweep-budgets", default="1,2,4,8")
    ap.add_argument("--sweep-slots", default="8,16,32")
    ap.add_argument("--sweep-adapters", default="random,gate_reuse,svd,fit",
                    help="adapter weights per sweep arm: random (the configuration), gate_reuse, svd, fit")
    ap.add_argument("--calib-steps", type=int, default=256, help="tokens of the calibration stream for --sweep-adapters fit")
    ap.add_argument("--stub-us", type=int, default=0,
                    help="attention stand-in of this many microseconds before each layer's router (widens the overlap window)")
    ap.add_argument("--copy-delay-us", type=int, default=0,
                    help="emulated slower storage tier: extra wait after every expert copy")
    ap.add_argument("--no-arms", action="store_true")
    ap.add_argument("--no-resident", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--oracle-threads", type=int, default=0, help="reference arm: BLAS threads (default: one)")
    ap.add_argument("--oracle-budget", type=int, default=-1, help="reference arm: prefetch budget (default: the configuration's, 1 if profiled)")
    ap.add_argument("--no-extra", action="store_true", help="skip the batched / DeepSeek-shaped legs and the targets block")
    ap.add_argument("--batched-steps", type=int, default=8)
    ap.add_argument("--dsvl2-steps", type=int, default=64)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU implementation")
        if args.sweep:
            run_sweep(args)
        else:
            run_ours(args)


if __name__ == "__main__":
    main()
