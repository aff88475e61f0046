"""End-to-end pins for the CPU oracle: the router-preserving guarantee, residency,
budget invariants and metric bounds on the tiny configuration. CPU only."""
import numpy as np
import pytest

import synth
from helpers import SynthWeights, make_ref
from oracle import ref_decode, ref_math as M, ref_policy as P


@pytest.fixture(scope="module")
def tiny():
    cfg = synth.get_config("tiny")
    tok = synth.zipf_tokens(cfg)
    H = synth.embedding_rows(cfg, tok[:, 0]).numpy()
    return cfg, SynthWeights(cfg), H


def run(cfg, wts, H, steps=24, nb=1, hint=None, **kw):
    ref = make_ref(cfg, weights=wts, **kw)
    outs, recs = [], []
    for s in range(steps):
        h, r = ref.step(H[s * nb:(s + 1) * nb], hint=None if hint is None else hint[s])
        outs.append(h); recs.append(r)
    return ref, np.stack(outs), recs


def test_router_preserving_guarantee(tiny):
    cfg, wts, H = tiny
    base_ref, base, base_recs = run(cfg, wts, H, slots=cfg.n_experts, policy=P.ON_DEMAND)
    hint = ref_decode.true_demand_trace(base_recs)
    arms = [dict(policy=P.ON_DEMAND), dict(policy=P.ADAPTER), dict(policy=P.ADAPTER, budget=4, slots=6),
            dict(policy=P.PRED0), dict(policy=P.HINT_TRACE, hint=hint), dict(policy=P.ADAPTER, plain_lru=True),
            dict(policy=P.ADAPTER, slots=2, budget=1), dict(policy=P.NAIVE, budget=2)]
    for kw in arms:
        _, out, recs = run(cfg, wts, H, **kw)
        assert np.array_equal(out, base), kw                       # bitwise: outputs never depend on the policy
        for a, b in zip(recs, base_recs):
            for ra, rb in zip(a, b):
                assert np.array_equal(ra.ids, rb.ids) and np.array_equal(ra.w, rb.w)


def test_naive_prefetch_replays_the_preceding_token(tiny):
    cfg, wts, H = tiny
    assert P.borda_ranking([[5, 2, 9]], 12) == [5, 2, 9]                   # one token: router rank order
    assert P.borda_ranking([[5, 2], [2, 7]], 12) == [2, 5, 7]              # 2: 1+2, 5: 2, 7: 1
    assert P.borda_ranking([[1, 0], [0, 1]], 4) == [0, 1]                  # tie -> lower id
    ref, _, recs = run(cfg, wts, H, policy=P.NAIVE, budget=2, slots=3)
    ev = ref.table.events
    assert not [e for e in ev if e[0] == 0 and e[2] == "PREFETCH"]          # no preceding token at step 0
    for (s, l, kind, e, slot) in ev:
        if kind == "PREFETCH":
            assert e in [int(x) for x in recs[s - 1][l].ids[0]]             # only experts the preceding token used there


def test_dropped_prefetch_requests_fall_back_to_demand(tiny):
    cfg, wts, H = tiny
    _, base, _ = run(cfg, wts, H, slots=cfg.n_experts, policy=P.ON_DEMAND)
    ref = make_ref(cfg, weights=wts)
    ref.drop_hook = lambda step, layer, e: (step + e) % 2 == 0
    outs = np.stack([ref.step(H[s:s + 1])[0] for s in range(24)])
    assert np.array_equal(outs, base)
    assert any(ev[2] == "DROPPED" for ev in ref.table.events)


def test_layer_math_matches_dense_definition(tiny):
    cfg, wts, H = tiny
    _, out, recs = run(cfg, wts, H, steps=3)
    # recompute step 2 densely, no slot table
    h = H[2].astype(np.float64)
    for l in range(cfg.n_layers):
        x = M.rmsnorm(h, np.ones(cfg.hidden), cfg.rms_eps)
        ids, w = M.route(M.router_logits(wts.router(l), x), cfg.top_k, True)
        y = sum(w[k] * M.swiglu_expert(*wts.expert(l, int(ids[k])), x) for k in range(cfg.top_k))
        h = h + y
        assert np.array_equal(ids, recs[2][l].ids[0])
    assert np.allclose(out[2][0], h, rtol=1e-12, atol=1e-14)
    assert abs(recs[0][0].w.sum() - 1) < 1e-12
    s = recs[0][0].scores
    assert abs(s.sum() - 1.0) < 1e-12 and list(recs[0][0].order) == list(M.rank_desc(s.astype(np.float32)))
    assert recs[0][cfg.n_layers - 1].scores is None           # L-1 adapters


def test_budget_and_exclusion_invariants(tiny):
    cfg, wts, H = tiny
    for budget in (1, 2, 3):
        ref = make_ref(cfg, weights=wts, budget=budget)
        for s in range(32):
            before = [set(ref.table.resident(l)) for l in range(cfg.n_layers)]
            _, recs = ref.step(H[s:s + 1])
            for l, rec in enumerate(recs[:-1]):
                assert len(rec.prefetch) <= budget                        # m_l <= M_max
                assert len(rec.issued) <= len(rec.prefetch)
                sc = rec.scores
                got = [sc[e] for e in rec.prefetch]
                assert got == sorted(got, reverse=True)                     # descending priority
        ev = ref.table.events
        # never prefetch an expert that already has a slot: between two PREFETCH/MISS of the same
        # (layer, expert) there is always an EVICT of it
        live = set()
        for (_, l, kind, e, _) in ev:
            if kind in ("MISS", "PREFETCH"):
                assert (l, e) not in live
                live.add((l, e))
            elif kind.startswith("EVICT"):
                live.discard((l, e))


def test_hint_trace_full_coverage_and_metrics(tiny):
    cfg, wts, H = tiny
    _, _, base_recs = run(cfg, wts, H, slots=cfg.n_experts, policy=P.ON_DEMAND)
    hint = ref_decode.true_demand_trace(base_recs)
    ref, _, recs = run(cfg, wts, H, policy=P.HINT_TRACE, hint=hint, budget=cfg.top_k)
    for step in recs:
        for l in range(1, cfg.n_layers):
            assert step[l].ready == 1.0                 # every needed expert had a slot at demand time
    assert [e for e in ref.table.events if e[2] == "MISS" and e[1] >= 1] == []
    od, _, od_recs = run(cfg, wts, H, policy=P.ON_DEMAND)
    assert od.table.stats.misses == ref.table.stats.misses + ref.table.stats.prefetch_issued
    # hint scores reach R@K = 1; random adapters stay within the M/K bound
    for step in base_recs:
        mass = np.zeros(cfg.n_experts); mass[step[1].ids[0]] = step[1].w[0]
        assert M.expert_recall_at_m(step[1].ids, mass, cfg.top_k, cfg.top_k) == 1.0
        assert M.expert_recall_at_m(step[1].ids, step[0].scores, 1, cfg.top_k) <= 1 / cfg.top_k


def test_batched_waves_preserve_outputs():
    cfg = synth.get_config("tiny").replace(batch=6)
    wts = SynthWeights(cfg)
    tok = synth.zipf_tokens(cfg, steps=4)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy()
    _, base, _ = run(cfg, wts, H, steps=4, nb=6, slots=cfg.n_experts, policy=P.ON_DEMAND)
    ref, out, recs = run(cfg, wts, H, steps=4, nb=6, slots=3)          # demand > slots -> waves
    assert max(r.n_waves for step in recs for r in step) > 1
    assert np.allclose(out, base, rtol=1e-13, atol=1e-15)
    # each sequence alone gives the same rows: tokens do not interact
    solo = make_ref(cfg, weights=wts, slots=cfg.n_experts, policy=P.ON_DEMAND)
    h1, _ = solo.step(H[2:3])
    assert np.allclose(h1[0], base[0][2], rtol=1e-13, atol=1e-15)
