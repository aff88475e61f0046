"""Edge and degenerate cases of the decode path on the GPU, each against the CPU oracle."""
import numpy as np
import pytest
import torch

import synth
from helpers import SynthWeights, make_ref
from oracle import ref_math as M, ref_policy as P

pytestmark = pytest.mark.gpu


def dev(a):
    t = torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float32).cuda()
    torch.cuda.synchronize()
    return t


def build(cfg, **kw):
    from paper_2607_24787_b200.build import build as b
    from paper_2607_24787_b200.synth_model import build_from_synth
    b()
    return build_from_synth(cfg, **kw)


def compare_run(cfg, steps=6, policy="adapter", tol=4e-5, **kw):
    m = build(cfg)
    wts = SynthWeights(cfg)
    nb = cfg.batch
    tok = synth.zipf_tokens(cfg, steps=steps)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(steps, nb, cfg.hidden)
    ref = make_ref(cfg, weights=wts, policy=policy, **kw)
    m.set_policy(policy)
    for s in range(steps):
        out = m.decode_step(dev(H[s]))
        m.synchronize()
        want, _ = ref.step(H[s])
        got = out.cpu().numpy().astype(np.float64)
        for t in range(nb):
            assert M.rel_linf(got[t], want[t]) < tol, (s, t)
    assert m.events() == ref.table.events
    m.check_invariants()
    st = m.stats()
    m.close()
    return st


def test_single_layer_has_no_adapter():
    st = compare_run(synth.get_config("tiny", n_layers=1))
    assert st["prefetch_issued"] == 0 and st["misses"] > 0


def test_top_k_equals_n_and_slots_equal_k():
    # every expert is used by every token: after the first step nothing is ever loaded again
    st = compare_run(synth.get_config("tiny", n_experts=4, top_k=4, slots=4, budget=2, adapter_rank=3))
    assert st["misses"] + st["prefetch_issued"] == 2 * 4          # each of the 8 experts is copied exactly once


def test_top_1_and_budget_zero():
    st = compare_run(synth.get_config("tiny", top_k=1, slots=1, budget=0))
    assert st["prefetch_issued"] == 0


def test_budget_larger_than_slots():
    st = compare_run(synth.get_config("tiny", slots=3, budget=9))
    assert st["prefetch_issued"] > 0


def test_max_hidden_bf16_and_odd_rank():
    compare_run(synth.get_config("qwen3", n_layers=2, n_experts=9, inter=40, top_k=2, slots=3, budget=1, adapter_rank=7),
                steps=4, tol=4e-4)


def test_shared_experts_batched_use_gemv_path():
    # shared experts + several sequences: the per-token GEMV kernel (fp32 activations), with waves
    cfg = synth.get_config("dsvl2", n_layers=2, n_experts=10, inter=64, top_k=3, slots=4, budget=1, batch=5)
    st = compare_run(cfg, steps=3, tol=4e-4)
    assert st["waves"] > 0


def test_full_batch_fp32():
    compare_run(synth.get_config("tiny", batch=64, slots=16, budget=2), steps=2)


def test_partial_host_store_repeats_layers():
    """A host that cannot pin the whole store keeps k layers of experts; layer l then reads layer l % k."""
    cfg = synth.get_config("tiny", n_layers=3)
    m = build(cfg, store_layers=2)

    class Repeating(SynthWeights):
        def expert(self, l, e):
            return super().expert(l % 2, e)

    ref = make_ref(cfg, weights=Repeating(cfg))
    tok = synth.zipf_tokens(cfg, steps=4)
    H = synth.embedding_rows(cfg, tok[:, 0]).numpy()
    for s in range(4):
        out = m.decode_step(dev(H[s:s + 1])); m.synchronize()
        want, _ = ref.step(H[s:s + 1])
        assert M.rel_linf(out.cpu().numpy(), want) < 4e-5
    assert m.events() == ref.table.events
    m.close()


def test_timing_knobs_do_not_change_results():
    """Attention stand-in and emulated storage delay only move time around."""
    cfg = synth.get_config("tiny")
    m = build(cfg)
    tok = synth.zipf_tokens(cfg, steps=4)
    H = synth.embedding_rows(cfg, tok[:, 0]).numpy()
    outs = []
    for stub, delay in ((0, 0), (200, 150)):
        m.cache_reset(); m.set_attention_stub_us(stub); m.set_copy_delay_us(delay)
        w = m.profile_window()
        run = []
        for s in range(4):
            out = m.decode_step(dev(H[s:s + 1])); m.synchronize()
            run.append(out.cpu().numpy())
        outs.append((np.stack(run), m.events(), w))
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    assert outs[1][2][0] > outs[0][2][0] + 150 and outs[1][2][1] > outs[0][2][1] + 100    # window and t_xfer grew
    m.close()


def test_profiled_budget_is_the_oracles_floor_of_window_over_transfer():
    """Window-aware budget (Section 3.3): the integer the profiler returns is the oracle's
    floor(W / t_xfer) of the very (W, t_xfer) it measured, with and without the attention stand-in,
    and a context created with budget = -1 runs with the oracle's max(1, raw) of its own profile."""
    cfg = synth.get_config("tiny")
    m = build(cfg)
    for stub in (0, 250, 0):
        m.set_attention_stub_us(stub)
        W, t, raw = m.profile_window()
        assert W > 0 and t > 0
        assert raw == M.window_budget(W, t), (stub, W, t, raw)
        assert m.get_profile() == (W, t, raw)
    # the stand-in makes the window hold at least one transfer here, so both branches of the clamp are seen
    m.set_attention_stub_us(2000)
    W, t, raw = m.profile_window()
    assert raw == M.window_budget(W, t) and raw >= 1
    m.close()
    auto = build(cfg, budget=-1)
    W, t, raw = auto.get_profile()
    assert raw == M.window_budget(W, t)
    assert auto.get_budget() == M.run_budget(W, t) == max(1, raw)
    auto.close()
    fixed = build(cfg, budget=3)
    assert fixed.get_budget() == 3
    with pytest.raises(Exception):
        fixed.get_profile()                      # never profiled
    fixed.close()


def test_device_side_wait_runs_out_reports_timeout_and_context_survives():
    """A wait inside the expert kernel has a limit: an arrival counter that is never bumped (the
    update is withheld on the host; the bytes themselves land) makes the kernel give up after the
    limit, set its status bit and return. The host reads SPM_ERR_TIMEOUT once; after a cache reset
    the same context decodes correctly again. Nothing on the GPU faults or spins for long."""
    import time
    from paper_2607_24787_b200 import binding as B
    if B.load() is None:
        pytest.skip("library missing")
    cfg = synth.get_config("tiny")
    m = build(cfg)
    try:
        m.set_device_wait(1)
    except B.SpmError:
        m.close()
        pytest.skip("stream-ordered memory writes are not available on this driver")
    m.set_device_wait_limit_us(3000)
    tok = synth.zipf_tokens(cfg, steps=3)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(3, 1, cfg.hidden)
    m.cache_reset()
    m.test_withhold_arrivals(1)                  # cleared by cache_reset, so set after it
    t0 = time.perf_counter()
    with pytest.raises(B.SpmError) as e:
        m.decode_step(dev(H[0]))
        m.synchronize()
    assert e.value.code == -4                    # SPM_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 1.9        # gave up after milliseconds, not after the 2 s default
    m.synchronize()                              # reported once
    # the same context, cache and counters reset, still computes what the oracle computes
    m.set_device_wait_limit_us(0)
    m.cache_reset()
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy="adapter")
    for s in range(3):
        out = m.decode_step(dev(H[s]))
        m.synchronize()
        want, _ = ref.step(H[s])
        assert M.rel_linf(out.cpu().numpy().astype(np.float64)[0], want[0]) < 4e-5
    assert m.events() == ref.table.events
    m.check_invariants()
    m.close()


def test_event_log_is_bounded_and_counters_do_not_depend_on_it():
    cfg = synth.get_config("tiny")
    tok = synth.zipf_tokens(cfg, steps=6)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(6, 1, cfg.hidden)
    m = build(cfg)
    runs = []
    for cap in (1 << 20, 7, 0):
        m.set_event_log_limit(cap)
        m.cache_reset()
        for s in range(6):
            m.decode_step(dev(H[s]))
        m.synchronize()
        runs.append((m.events(), m.stats()))
    full, st_full = runs[0]
    assert st_full["events_dropped"] == 0 and len(full) > 7
    for (ev, st), cap in zip(runs[1:], (7, 0)):
        assert ev == full[:cap] and st["events_dropped"] == len(full) - cap
        for k in ("hits", "misses", "evictions", "prefetch_issued", "wasted", "touches"):
            assert st[k] == st_full[k], k
    m.close()


def test_host_deadline_returns_timeout_and_context_survives():
    """The routing handshake has a host-side deadline: with the compute stream kept busy by unrelated
    work the call gives up with SPM_ERR_TIMEOUT instead of spinning; nothing on the GPU is disturbed."""
    from paper_2607_24787_b200 import binding as B
    cfg = synth.get_config("tiny")
    m = build(cfg)
    h = dev(np.ones((1, cfg.hidden)))
    a = torch.randn(8192, 8192, device="cuda")
    B.spm_set_deadline_ms(m.ctx, 1)
    with torch.cuda.stream(m.compute):
        for _ in range(40):                      # roughly 50 ms of matmuls queued ahead of the router kernel
            a = a @ a
            a = a / a.norm()
    with pytest.raises(B.SpmError) as e:
        m.decode_step(h)
    assert e.value.code == -4
    torch.cuda.synchronize()
    B.spm_set_deadline_ms(m.ctx, 5000)
    m.cache_reset()
    ref = make_ref(cfg, weights=SynthWeights(cfg))
    out = m.decode_step(h)
    m.synchronize()
    want, _ = ref.step(np.ones((1, cfg.hidden)))
    assert M.rel_linf(out.cpu().numpy(), want) < 4e-5
    m.close()


def test_read_bandwidth_probe_and_its_limits():
    cfg = synth.get_config("qwen3", n_layers=2, slots=24)          # 2 x 24 x 9 MiB = 432 MiB of pools
    m = build(cfg)
    before = [list(m.slot_table(l)) for l in range(cfg.n_layers)]
    g = m.measure_read_bandwidth(1 << 40, reps=3)                    # clamped to the pools
    assert 1000.0 < g < 12000.0, g                                   # GB/s: above PCIe, below any HBM3e figure
    assert before == [list(m.slot_table(l)) for l in range(cfg.n_layers)]
    with pytest.raises(Exception):
        m.measure_read_bandwidth(1 << 20)                            # too small to get past L2
    m.close()


def test_cache_checkpoint_resumes_a_run_bit_for_bit():
    # export the cache state mid-run, import it into a fresh context: the rest of the run gives the
    # same outputs, events and slot tables as the uninterrupted one and as the oracle
    cfg = synth.get_config("tiny", slots=5, budget=2)
    steps, half = 16, 7
    tok = synth.zipf_tokens(cfg, steps=steps)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(steps, 1, cfg.hidden)
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy="adapter")
    a = build(cfg)
    outs = []
    for s in range(steps):
        if s == half:
            state = a.cache_export()
            mark = len(a.events())
        outs.append(a.decode_step(dev(H[s])))
        a.synchronize()
        want, _ = ref.step(H[s])
        assert M.rel_linf(outs[-1].cpu().numpy().astype(np.float64)[0], want[0]) < 4e-5
    assert a.events() == ref.table.events
    b = build(cfg)
    b.cache_import(state)
    assert b.stats()["h2d_bytes"] == 0 and b.events() == []
    for s in range(half, steps):
        out = b.decode_step(dev(H[s]))
        b.synchronize()
        assert np.array_equal(out.cpu().numpy(), outs[s].cpu().numpy()), s
    assert b.events() == a.events()[mark:]
    assert [list(b.slot_table(l)) for l in range(cfg.n_layers)] == [list(a.slot_table(l)) for l in range(cfg.n_layers)]
    with pytest.raises(Exception):
        b.cache_import(state[:-1])
    a.close(); b.close()


def test_non_finite_hidden_row_is_reported_not_propagated_silently():
    from paper_2607_24787_b200 import binding as B
    cfg = synth.get_config("tiny")
    m = build(cfg)
    tok = synth.zipf_tokens(cfg, steps=2)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(2, 1, cfg.hidden)
    bad = H[0].copy()
    bad[0, 7] = np.inf
    m.decode_step(dev(bad))
    with pytest.raises(B.SpmError) as e:
        m.synchronize()
    assert e.value.code == -7
    # reported once; the context keeps working
    m.cache_reset()
    out = m.decode_step(dev(H[1]))
    m.synchronize()
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy="adapter")
    want, _ = ref.step(H[1])
    assert M.rel_linf(out.cpu().numpy().astype(np.float64)[0], want[0]) < 4e-5
    m.close()


def test_long_run_with_changing_policies_and_wait_modes_stays_router_preserving():
    """800 decode steps on one context while the policy, the budget, the way the FFN waits for its copies
    and the fault injection on prefetch requests change every 40 steps: every step's output equals, bit for
    bit, the output of a context that holds all experts (Section 3.1: prediction never changes routing or
    outputs), the slot table's invariants hold throughout, and the counters add up."""
    from paper_2607_24787_b200 import binding as B
    cfg = synth.get_config("tiny", n_layers=3, n_experts=12, slots=5, budget=2)
    steps, span = 800, 40
    tok = synth.zipf_tokens(cfg, steps=steps)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(steps, 1, cfg.hidden)
    full = build(cfg, slots=cfg.n_experts, budget=0)
    full.set_policy("on_demand")
    want = []
    for s in range(steps):
        want.append(full.decode_step(dev(H[s])))
    full.synchronize()
    want = [w.cpu().numpy() for w in want]
    full.close()
    m = build(cfg)
    try:
        can_wait = True
        try:
            m.set_device_wait(1); m.set_device_wait(0)
        except B.SpmError:
            can_wait = False
        policies = ["adapter", "on_demand", "naive", "pred0", "adapter"]
        outs = []
        for s in range(steps):
            if s % span == 0:
                phase = s // span
                m.synchronize()
                m.check_invariants()
                m.set_policy(policies[phase % len(policies)])
                m.set_budget(phase % 4)
                m.set_drop_modulo(3 if phase % 3 == 2 else 0)
                if can_wait:
                    m.set_device_wait(phase % 2)
            outs.append(m.decode_step(dev(H[s])))
        m.synchronize()
        for s in range(steps):
            assert np.array_equal(outs[s].cpu().numpy(), want[s]), s
        st = m.stats()
        assert st["hits"] + st["misses"] == steps * cfg.n_layers * cfg.top_k
        assert st["steps"] == steps and st["prefetch_issued"] > 0 and st["dropped"] > 0
        m.check_invariants()
    finally:
        m.close()


def test_ffn_kernel_probe_in_all_launch_modes_leaves_the_context_usable():
    """`spm_time_ffn_kernel` (the measurement aid behind the bench's roofline): plain and chained launches,
    each also replayed from a CUDA graph, return positive times and an in-kernel window; an expert without a
    slot is refused; a decode step afterwards still matches the oracle."""
    from paper_2607_24787_b200 import binding as B
    cfg = synth.get_config("tiny", n_layers=2)
    m = build(cfg, slots=cfg.n_experts, budget=0)
    try:
        m.set_policy("on_demand")
        x = torch.randn(cfg.hidden, device="cuda")
        w = torch.full((cfg.top_k,), 1.0 / cfg.top_k, device="cuda")
        ids = np.stack([np.arange(cfg.top_k, dtype=np.int32) + (i % 3) for i in range(24)])
        with pytest.raises(B.SpmError):
            m.time_ffn_kernel(0, x, ids, w, chained=0)         # nothing resident yet: the probe loads nothing
        for l in range(cfg.n_layers):
            m.prefetch_async(l, np.arange(cfg.n_experts, dtype=np.int32))
        m.synchronize()
        for mode in (0, 1, 2, 3):
            us, win = m.time_ffn_kernel(0, x, ids, w, chained=mode)
            assert 0.0 < us < 1e4 and 0.0 < win < 1e4, (mode, us, win)
        tok = synth.zipf_tokens(cfg, steps=2)
        H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(2, 1, cfg.hidden)
        ref = make_ref(cfg, weights=SynthWeights(cfg), policy="on_demand", slots=cfg.n_experts, budget=0)
        for s in range(2):
            out = m.decode_step(dev(H[s]))
            m.synchronize()
            want, _ = ref.step(H[s])
            assert M.rel_linf(out.cpu().numpy().astype(np.float64)[0], want[0]) < 4e-5
    finally:
        m.close()
