"""Host-free decode steps (every expert resident: no routing result can change what the prefetch
controller does, so a step is enqueued without a host turn and the slot table's bookkeeping is
replayed from a device-written trace). Outputs, cache events and statistics must equal the CPU
oracle's and, bit for bit, those of the host-driven path."""
import numpy as np
import pytest
import torch

import synth
from helpers import SynthWeights, make_ref
from oracle import ref_math as M

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-5, "bf16": 1e-4, "q4": 1e-4}

SHAPES = {
    "tiny": synth.get_config("tiny", slots=16),
    "tiny_b3": synth.get_config("tiny", slots=16, batch=3),
    "ds_small": synth.get_config("dsvl2", n_layers=3, n_experts=16, inter=224, slots=16, budget=2),
    "q4_qw": synth.get_config("qwen3_q4", n_layers=2, n_experts=24, inter=96, slots=24, budget=3),
    "odd": synth.get_config("tiny", hidden=384, inter=50, n_experts=11, top_k=3, adapter_rank=5, slots=11, seed=7),
}


def build(cfg, **kw):
    from paper_2607_24787_b200.build import build as b
    from paper_2607_24787_b200.synth_model import build_from_synth
    b()
    return build_from_synth(cfg, **kw)


def rows(cfg, steps):
    tok = synth.zipf_tokens(cfg, steps=steps)
    return synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(steps, cfg.batch, cfg.hidden)


def preload(cfg, m, ref=None):
    everything = list(range(cfg.n_experts))
    for l in range(cfg.n_layers):
        assert m.prefetch_async(l, everything) == cfg.n_experts
        if ref is not None:
            for e, s in ref.table.prefetch(l, everything, [], set()):
                ref._copy_in(l, e, s)


def run(m, H, sync_every=0):
    outs = []
    for s in range(H.shape[0]):
        h = torch.as_tensor(H[s], dtype=torch.float32).cuda()
        torch.cuda.synchronize()
        outs.append(m.decode_step(h))
        if sync_every and (s + 1) % sync_every == 0:
            m.synchronize()
    m.synchronize()
    return [o.cpu().numpy() for o in outs]


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("policy", ["adapter", "on_demand", "naive", "pred0"])
def test_host_free_steps_match_oracle_and_host_driven_path(name, policy):
    cfg = SHAPES[name]
    steps = 20                      # more than the trace ring holds, none synchronised in between
    H = rows(cfg, steps)
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy=policy)
    m = build(cfg)
    m.set_policy(policy)
    preload(cfg, m, ref)
    got = run(m, H)
    st = m.stats()
    assert st["host_free_steps"] == steps and st["misses"] == 0 and st["steps"] == steps
    for s in range(steps):
        want, _ = ref.step(H[s])
        for t in range(cfg.batch):
            assert M.rel_linf(got[s][t].astype(np.float64), want[t]) < 4 * TOL[cfg.dtype], (s, t)
    assert m.events() == ref.table.events
    assert st["hits"] == ref.table.stats.hits and st["touches"] == ref.table.stats.touches
    slot_tables = [list(m.slot_table(l)) for l in range(cfg.n_layers)]
    m.close()

    # the host-driven path on the same inputs: same bits, same events, same statistics
    m2 = build(cfg)
    m2.set_host_free(0)
    m2.set_policy(policy)
    preload(cfg, m2)
    got2 = run(m2, H, sync_every=1)
    st2 = m2.stats()
    assert st2["host_free_steps"] == 0
    for s in range(steps):
        assert np.array_equal(got[s], got2[s]), s
    assert m2.events() == ref.table.events
    for k in ("hits", "misses", "touches", "planned", "steps", "tokens", "recall_count", "ready_count"):
        assert st[k] == st2[k], k
    assert st["recall_sum"] == st2["recall_sum"] and st["ready_sum"] == st2["ready_sum"]
    assert slot_tables == [list(m2.slot_table(l)) for l in range(cfg.n_layers)]
    m2.close()


def test_host_free_state_ends_with_cache_reset_and_resumes():
    cfg = SHAPES["tiny"]
    H = rows(cfg, 12)
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy="adapter")
    m = build(cfg)
    preload(cfg, m, ref)
    a = run(m, H[:4])
    assert m.stats()["host_free_steps"] == 4
    m.cache_reset()
    ref.table.reset()
    ref.storage = [dict() for _ in range(cfg.n_layers)]
    b = run(m, H[4:8])                       # pools empty again: host-driven, with misses
    st = m.stats()
    assert st["host_free_steps"] == 0 and st["misses"] > 0
    wants = [ref.step(H[s])[0] for s in range(4, 8)]
    for s in range(4):
        assert M.rel_linf(b[s][0].astype(np.float64), wants[s][0]) < 4e-5
    assert m.events() == ref.table.events
    # fill what is still missing, then the state is entered again
    for l in range(cfg.n_layers):
        missing = [e for e in range(cfg.n_experts) if e not in m.slot_table(l)]
        assert m.prefetch_async(l, missing) == len(missing)
        for e, s in ref.table.prefetch(l, missing, [], set()):
            ref._copy_in(l, e, s)
    before = m.stats()["host_free_steps"]
    c = run(m, H[8:12])
    assert m.stats()["host_free_steps"] == before + 4
    for s in range(4):
        want, _ = ref.step(H[8 + s])
        assert M.rel_linf(c[s][0].astype(np.float64), want[0]) < 4e-5
    assert m.events() == ref.table.events
    m.close()


def test_calls_between_host_free_steps_see_replayed_state():
    # a stand-alone call after un-synchronised host-free steps must find the table as the oracle has it
    cfg = SHAPES["tiny"]
    H = rows(cfg, 6)
    ref = make_ref(cfg, weights=SynthWeights(cfg), policy="adapter")
    m = build(cfg)
    preload(cfg, m, ref)
    for s in range(5):
        h = torch.as_tensor(H[s], dtype=torch.float32).cuda()
        torch.cuda.synchronize()
        m.decode_step(h)
        ref.step(H[s])
    assert len(m.events()) == len(ref.table.events)        # no synchronize in between: the call replays
    assert m.events() == ref.table.events
    m.close()


TC_CASES = {
    "wide": synth.get_config("qwen3", n_layers=2, hidden=1280, n_experts=16, inter=384, top_k=3, slots=16, budget=2, batch=64),
    "many_tokens": synth.get_config("qwen3", n_layers=3, hidden=512, n_experts=8, inter=128, top_k=2, slots=8, budget=1, batch=64),
    "ragged_batch": synth.get_config("qwen3", n_layers=2, hidden=256, n_experts=24, inter=256, top_k=4, slots=24, budget=2, batch=17),
    "q4_wide": synth.get_config("qwen3_q4", n_layers=2, hidden=1280, n_experts=16, inter=384, top_k=3, slots=16, budget=2, batch=64),
}


@pytest.mark.parametrize("case", list(TC_CASES))
def test_host_free_tensor_core_path_equals_host_driven(case):
    # batched steps: the wave plan (token rows sorted by expert, units, combine map) is built by a
    # kernel instead of the host; the grouped tcgen05 FFN must see the same plan
    cfg = TC_CASES[case]
    steps = 11
    H = rows(cfg, steps)
    results = []
    for host_free in (1, 0):
        m = build(cfg)
        m.set_host_free(host_free)
        m.set_policy("adapter")
        preload(cfg, m)
        outs = run(m, H, sync_every=0 if host_free else 1)
        st = m.stats()
        assert st["host_free_steps"] == (steps if host_free else 0) and st["misses"] == 0
        results.append((outs, m.events(), {k: st[k] for k in ("hits", "touches", "steps", "tokens", "recall_sum", "ready_sum")}))
        m.close()
    (a, ev_a, st_a), (b, ev_b, st_b) = results
    for s in range(steps):
        assert np.array_equal(a[s], b[s]), s
    assert ev_a == ev_b and st_a == st_b


@pytest.mark.parametrize("name", ["tiny", "ds_small", "tiny_b3"])
def test_graph_replay_gives_the_same_bits_and_bookkeeping(name):
    cfg = SHAPES[name]
    steps = 24                      # three laps of the trace ring: every slot's graph is captured, then replayed
    H = rows(cfg, steps)
    results = []
    for replay in (1, 0):
        m = build(cfg)
        m.set_graph_replay(replay)
        preload(cfg, m)
        outs = run(m, H)
        st = m.stats()
        assert st["host_free_steps"] == steps
        results.append((outs, m.events(), {k: st[k] for k in ("hits", "touches", "steps", "tokens", "kernel_launches", "ffn_launches", "recall_sum")}))
        m.close()
    (a, ev_a, st_a), (b, ev_b, st_b) = results
    for s in range(steps):
        assert np.array_equal(a[s], b[s]), s
    assert ev_a == ev_b and st_a == st_b
