"""The benchmark's multi-rank logic on CPU: 2 gloo ranks, independent token streams per rank,
max-over-ranks time and summed tokens (no collective on the data path)."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    import bench, synth
    rank, local, world = bench.dist_setup("gloo")
    cfg = synth.get_config("tiny")
    tok, H = bench.hidden_rows(cfg, 16, stream=rank)
    bench.barrier(world)
    t, n = bench.aggregate(10.0 + 5.0 * rank, 16 * cfg.batch, world)
    print(json.dumps({"rank": rank, "world": world, "t": t, "n": n, "tok": tok[:, 0].tolist(), "shape": list(H.shape)}))
""") % ROOT


def _run_two_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs, errs = [], []
    for p in procs:
        try:
            out, err = p.communicate(timeout=180)
        except subprocess.TimeoutExpired:
            p.kill()
            out, err = p.communicate()
            err += "\n(timed out)"
        if p.returncode != 0:
            errs.append(err[-2000:])
        else:
            outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    return outs, errs


def test_two_gloo_ranks_shard_by_sequence():
    # the rendezvous port is picked by binding and releasing it, so another process can take it in
    # between: a failed rendezvous is retried on a fresh port
    for attempt in range(3):
        outs, errs = _run_two_ranks()
        if not errs:
            break
    assert not errs, errs
    outs.sort(key=lambda o: o["rank"])
    assert [o["world"] for o in outs] == [2, 2]
    assert all(o["t"] == 15.0 for o in outs)            # max over ranks
    assert all(o["n"] == 32 for o in outs)              # tokens of all ranks
    assert outs[0]["tok"] != outs[1]["tok"]             # every rank decodes its own sequence
    assert outs[0]["shape"] == [16, 1, 256]


def test_reference_arm_prints_contract_line():
    """`--impl reference` (the CPU oracle) runs without a GPU and prints one JSON line."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "4", "--warmup", "3"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = __import__("json").loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "tokens/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # under torchrun only rank 0 prints; the others exit 0 without work
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_line_and_results_formatter(tmp_path):
    """`bench.py --impl reference` (the CPU oracle, timed) prints one JSON line that carries the contract's keys and
    the same declarative `config` block as the GPU arm; `results_tables.py` turns it into text."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "tiny", "--steps", "3", "--warmup", "3"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
              "dtype", "data", "config", "cpu_baseline", "e2e", "impl"):
        assert k in d, k
    assert d["impl"] == "reference" and d["steps"] == 3 and d["value"] > 0 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("tiny:") and "budget_rule" in d["config"]
    f = tmp_path / "ref.json"
    f.write_text(line + "\n")
    txt = subprocess.run([sys.executable, os.path.join(root, "results_tables.py"), str(f)], capture_output=True, text=True, timeout=60)
    assert txt.returncode == 0 and "Reference arm" in txt.stdout


def test_results_formatter_on_a_gpu_arm_line(tmp_path):
    """`results_tables.py` on a line shaped like the GPU arm's (every block the default run emits): arms, targets
    with the paper-regime arms, the kernels' rooflines per workload, the resident legs and the CPU baseline."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    arm = {"tok_s": 17.1, "stall_us_per_layer": 1180.0, "hit_rate": 0.16, "ready_recall": 0.16, "copies_per_token": 322.7,
           "prefetch_used": 0, "prefetch_wasted": 0, "h2d_gb_s_avg": 52.2, "expert_recall_at_budget": None, "steps": 8}
    roof = {"bound": "hbm", "kernel": "ffn_gemv_kernel", "achieved": 5600.0, "peak": 6551.0, "unit": "GB/s", "frac": 0.855, "traffic": 76.6e6,
            "peak_source": "of measured", "algorithmic_bytes_per_launch": 75497472.0, "us_per_launch": 13.5, "us_per_launch_serialized": 16.5,
            "frac_serialized": 0.70, "us_per_launch_event_pair_each": 20.1, "in_kernel_window_us": 12.7, "read_only_stream_gb_s": 7150.0}
    regime = {"attention_stub_us": 354, "steps_per_arm": 32, "window_us": 377.0, "t_xfer_us": 177.0, "budget_raw": 2, "budget": 2}
    for k, g in (("on_demand", 0.0), ("adapter_gate_reuse", 0.21)):
        regime[k] = {"tok_s": 12.8 * (1 + g), "stall_us_per_layer": 1230.0, "ready_recall": 0.13, "expert_recall_at_budget": None,
                     "gain_over_on_demand": g}
    line = {
        "metric": "decode tokens/s with offloaded experts", "value": 15.5, "unit": "tokens/s", "n_gpus": 1, "steps": 256, "warmup": 8,
        "ms_per_step": 64.3, "config": {"workload": "qwen3: L48"}, "profile": {"window_us": 26.3, "t_xfer_us": 177.0, "budget_raw": 0, "budget": 1},
        "clocks": {"sm_mhz": 1965.0, "reasons": []}, "e2e": {"value": 15.4}, "gpu_launches": 24832, "roofline": roof,
        "main_arm": dict(arm, tok_s=15.5), "arms": {"on_demand": arm},
        "h2d": {"expert_copies_gb_s": 53.8, "pinned_peak_gb_s": 55.6, "frac": 0.967},
        "targets": {"on_demand": {"stall_us_per_layer": 1180.0, "tok_s": 17.1},
                    "adapter_gate_reuse": {"stall_us_per_layer": 1094.0, "tok_s": 17.4, "expert_recall_at_budget": 0.125},
                    "exposed_below_on_demand": {"adapter_gate_reuse": True}, "paper_regime": regime},
        "configs": {"batched": {"workload": "batched: L48", "profile": {"window_us": 117.0, "t_xfer_us": 177.0},
                                "offloaded": dict(arm, tok_s=81.0), "offloaded_device_wait": {"tok_s": 81.6},
                                "roofline_wave": dict(roof, kernel="ffn_grouped_kernel"), "roofline": dict(roof, kernel="ffn_grouped_kernel"),
                                "resident_host_free_tok_s": 6020.0},
                    "dsvl2": {"error": "not run"}},
        "resident": {"tok_s": 449.0, "host_free_on_demand": {"tok_s_untimed_launches": 805.0, "tok_s_untimed_graph_replay": 865.0, "us_per_layer": 26.3,
                                                             "ffn_window_us": 14.4, "router_window_us": 8.7, "idle_between_kernels_us_per_layer": 3.1,
                                                             "hbm_bound_tok_s": 1808.0},
                     "host_free_adapter": {"tok_s_untimed_graph_replay": 827.0}},
        "cpu_baseline": {"value": 1.1, "cores": 1, "per_step": [0.9, 1.1, 1.15], "all_host_cores": {"value": 3.8, "cores": 16}, "sample": "3 steps"},
    }
    f = tmp_path / "gpu.json"
    f.write_text(json.dumps(line) + "\n")
    txt = subprocess.run([sys.executable, os.path.join(root, "results_tables.py"), str(f)], capture_output=True, text=True, timeout=60)
    assert txt.returncode == 0, txt.stderr[-2000:]
    for needle in ("adapter_gate_reuse", "+21.0 %", "ffn_grouped_kernel", "batched (one wave)", "CPU oracle", "producer warps", "error: not run"):
        assert needle in txt.stdout, needle
