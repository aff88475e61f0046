#!/usr/bin/env python
"""Turns bench.py output (JSON lines, one per run) into the markdown tables of RESULTS.md.

    python bench.py > default.json
    python bench.py --config sweep --sweep --steps 256 > sweep.json
    python results_tables.py default.json sweep.json > tables.md

Every table of RESULTS.md is the output of this script on the JSON lines named there; nothing is
typed in by hand. Lines that are not JSON objects are skipped.
"""
from __future__ import annotations

import json
import sys


def fmt(v, nd=2):
    if v is None:
        return ""
    if isinstance(v, bool):
        return "yes" if v else "no"
    if isinstance(v, int):
        return str(v)
    return f"{v:.{nd}f}"


def table(header, rows):
    out = ["| " + " | ".join(header) + " |", "|" + "---|" * len(header)]
    out += ["| " + " | ".join(r) + " |" for r in rows]
    return "\n".join(out)


def sweep_tables(d):
    print(f"### Sweep: {d['sweep']}, attention stand-in {d.get('attention_stub_us', 0)} us\n")
    print(f"Window W = {fmt(d['window_us'], 1)} us, t_xfer = {fmt(d['t_xfer_us'], 1)} us, floor(W / t_xfer) = {d['budget_raw']}.\n")
    hdr = ["slots", "M_max", "policy", "tok/s", "stall us/layer", "hit rate", "ReadyRecall", "ExpertRecall@M", "copies/token",
           "prefetched", "used", "wasted", "late"]
    rows = []
    for c in d["cells"]:
        rows.append([str(c["slots"]), str(c["budget"]), c["policy"], fmt(c["tok_s"]), fmt(c["stall_us_per_layer"], 1), fmt(c["hit_rate"], 3),
                     fmt(c["ready_recall"], 3), fmt(c["expert_recall_at_budget"], 3), fmt(c["copies_per_token"], 1),
                     str(c["prefetch_issued"]), str(c["prefetch_used"]), str(c["prefetch_wasted"]), str(c["late_arrivals"])])
    print(table(hdr, rows))
    cov = [c for c in d["cells"] if c.get("expert_recall_at_half_k_k_k_plus_2")]
    if cov:
        print("\nNext-layer coverage of the ranking (ExpertRecall at M = K/2, K, K+2; model-level, independent of slots and budget):\n")
        seen, rows = set(), []
        for c in cov:
            if c["policy"] in seen:
                continue
            seen.add(c["policy"])
            r = c["expert_recall_at_half_k_k_k_plus_2"]
            rows.append([c["policy"], fmt(r[0], 3), fmt(r[1], 3), fmt(r[2], 3)])
        print(table(["policy", "R@K/2", "R@K", "R@K+2"], rows))
    print()


def roofline_row(name, r):
    return [name, r.get("kernel", ""), fmt(r.get("algorithmic_bytes_per_launch", 0) / 1e6, 1), fmt(r.get("us_per_launch"), 1),
            fmt(r.get("achieved"), 0), fmt(r.get("frac"), 3), fmt(r.get("us_per_launch_serialized"), 1), fmt(r.get("frac_serialized"), 3),
            fmt(r.get("us_per_launch_graph_plain"), 1), fmt(r.get("frac_graph_plain"), 3),
            fmt(r.get("us_per_launch_event_pair_each"), 1), fmt(r.get("in_kernel_window_us"), 1)]


def bench_tables(d):
    cfg = d["config"]["workload"]
    print(f"### `{cfg}` — {d['steps']} steps, {d['warmup']} warm-up\n")
    p = d.get("profile", {})
    print(f"value = {fmt(d['value'])} {d['unit']} (adapter policy), end to end through host buffers {fmt(d['e2e']['value'])}; "
          f"{fmt(d['ms_per_step'], 2)} ms per step; W = {fmt(p.get('window_us'), 1)} us, t_xfer = {fmt(p.get('t_xfer_us'), 1)} us, "
          f"raw budget {p.get('budget_raw')}, budget used {p.get('budget')}; kernels launched in the timed region: {d.get('gpu_launches')}; "
          f"SM clock {d.get('clocks', {}).get('sm_mhz')} MHz, reasons {d.get('clocks', {}).get('reasons')}.\n")
    arms = {"adapter (the configuration's random adapters; `value`)": d.get("main_arm")}
    arms.update(d.get("arms", {}))
    rows = []
    for k, a in arms.items():
        if not a:
            continue
        rows.append([k, fmt(a["tok_s"]), fmt(a["stall_us_per_layer"], 1), fmt(a["hit_rate"], 3), fmt(a["ready_recall"], 3),
                     fmt(a["copies_per_token"], 1), f"{a['prefetch_used']} / {a['prefetch_wasted']}", fmt(a["h2d_gb_s_avg"], 1)])
    print(table(["arm", "tok/s", "stall us/layer", "hit rate", "ReadyRecall", "copies/token", "prefetch used / wasted", "H2D GB/s (avg)"], rows))
    if "h2d" in d:
        h = d["h2d"]
        print(f"\nExpert copies {fmt(h['expert_copies_gb_s'], 1)} GB/s = {fmt(h['frac'], 3)} of the pinned peak measured in the same run "
              f"({fmt(h['pinned_peak_gb_s'], 1)} GB/s).")
    t = d.get("targets")
    if t and "error" not in t:
        print("\nExposed transfer time per layer against on-demand loading at the same slots:\n")
        rows = [[k, fmt(v["stall_us_per_layer"], 1), fmt(v["tok_s"]), fmt(v.get("expert_recall_at_budget"), 3),
                 fmt(t["exposed_below_on_demand"].get(k)) if k != "on_demand" else ""]
                for k, v in t.items() if isinstance(v, dict) and "stall_us_per_layer" in v]
        print(table(["arm", "stall us/layer", "tok/s", "ExpertRecall@M", "below on-demand"], rows))
    pr = (t or {}).get("paper_regime")
    if pr and "error" not in pr:
        print(f"\nWith an attention stand-in of {pr['attention_stub_us']} us per layer (window {fmt(pr['window_us'], 0)} us = "
              f"{fmt(pr['window_us'] / pr['t_xfer_us'], 2)} transfers, the paper's regime; budget = floor(W / t_xfer) = {pr['budget_raw']}), "
              f"{pr['steps_per_arm']} steps per arm:\n")
        rows = [[k, fmt(v["tok_s"]), fmt(v["stall_us_per_layer"], 1), fmt(v.get("ready_recall"), 3), fmt(v.get("expert_recall_at_budget"), 3),
                 f"{100 * v['gain_over_on_demand']:+.1f} %"] for k, v in pr.items() if isinstance(v, dict) and "tok_s" in v]
        print(table(["arm", "tok/s", "stall us/layer", "ReadyRecall", "ExpertRecall@M", "against on-demand"], rows))
    print("\nExpert-FFN kernels against the measured HBM copy bandwidth:\n")
    rows = [roofline_row(cfg.split(":")[0], d["roofline"])]
    for name, leg in (d.get("configs") or {}).items():
        if "error" in leg:
            rows.append([name, "error: " + leg["error"][:60]] + [""] * 10)
            continue
        if "roofline_wave" in leg:
            rows.append(roofline_row(name + " (one wave)", leg["roofline_wave"]))
        rows.append(roofline_row(name + (" (all resident)" if "roofline_wave" in leg else ""), leg["roofline"]))
    print(table(["workload", "kernel", "MB per launch", "us per launch", "GB/s", "of peak", "us serialized", "of peak",
                 "us plain, replayed from a CUDA graph", "of peak", "us event pair each", "in-kernel window us"], rows))
    r = d["roofline"]
    print(f"\n(peak {fmt(r['peak'], 0)} GB/s {r.get('peak_source', '')}; read-only streaming rate of the device {fmt(r.get('read_only_stream_gb_s'), 0)} GB/s; "
          + (f"ncu DRAM traffic per launch {fmt(r['traffic'] / 1e6, 1)} MB.)" if r.get("traffic") else "no ncu traffic figure for this workload.)"))
    res = d.get("resident")
    if res and "error" not in res:
        hf = res.get("host_free_on_demand", {})
        print(f"\nAll experts resident: {fmt(res['tok_s'], 0)} tok/s host-driven; host-free steps {fmt(hf.get('tok_s_untimed_launches'), 0)} tok/s launch by launch, "
              f"{fmt(hf.get('tok_s_untimed_graph_replay'), 0)} replayed from CUDA graphs (adapter policy "
              f"{fmt(res.get('host_free_adapter', {}).get('tok_s_untimed_graph_replay'), 0)}); per layer {fmt(hf.get('us_per_layer'), 1)} us = FFN window "
              f"{fmt(hf.get('ffn_window_us'), 1)} + routing kernel {fmt(hf.get('router_window_us'), 1)} + idle {fmt(hf.get('idle_between_kernels_us_per_layer'), 1)}; "
              f"HBM bound {fmt(hf.get('hbm_bound_tok_s'), 0)} tok/s.")
    for name, leg in (d.get("configs") or {}).items():
        if "error" in leg:
            continue
        o = leg["offloaded"]
        print(f"\n`{leg['workload']}`: offloaded {fmt(o['tok_s'], 1)} tok/s (adapter policy, {o['steps']} steps, stall {fmt(o['stall_us_per_layer'], 0)} us per layer, "
              f"{fmt(o['copies_per_token'], 1)} copies per token, H2D {fmt(o['h2d_gb_s_avg'], 1)} GB/s); all resident, host-free "
              f"{fmt(leg.get('resident_host_free_tok_s'), 0)} tok/s; W = {fmt(leg['profile']['window_us'], 1)} us, t_xfer = {fmt(leg['profile']['t_xfer_us'], 1)} us.")
        dw = leg.get("offloaded_device_wait")
        if dw and "error" not in dw:
            print(f"With the kernel's producer warps waiting for the copies themselves: {fmt(dw['tok_s'], 1)} tok/s.")
    c = d.get("cpu_baseline")
    if c:
        print(f"\nCPU oracle: {fmt(c['value'], 3)} tok/s on {c['cores']} thread(s) (per step {[round(x, 3) for x in c.get('per_step', c.get('repeats', []))]}); "
              f"{fmt(c.get('all_host_cores', {}).get('value'), 3)} tok/s with {c.get('all_host_cores', {}).get('cores')} threads. {c['sample']}.")
    print()


def main():
    for path in sys.argv[1:]:
        for line in open(path):
            line = line.strip()
            if not line.startswith("{"):
                continue
            try:
                d = json.loads(line)
            except ValueError:
                continue
            if "sweep" in d:
                sweep_tables(d)
            elif d.get("impl") == "reference":
                print(f"Reference arm (CPU oracle): {fmt(d['value'], 3)} {d['unit']}, {fmt(d['ms_per_step'], 0)} ms per step; {d['cpu_baseline']['sample']}.\n")
            elif "roofline" in d:
                bench_tables(d)


if __name__ == "__main__":
    main()
