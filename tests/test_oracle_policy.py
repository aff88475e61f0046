"""Pins for oracle/ref_policy.py: brute-force selection, an independent LRU, closed-form
hit rates, invariants of Section 3.3 and the on-demand / perfect-knowledge identity. CPU only."""
from collections import OrderedDict

import numpy as np
import pytest

from oracle import ref_policy as P

rng = np.random.default_rng(99)


# ---------------------------------------------------------------- selection (Section 3.3)
def test_select_bruteforce_and_invariants():
    for _ in range(200):
        n = int(rng.integers(2, 40))
        s = np.round(rng.normal(size=n), 1)                 # ties on purpose
        resident = set(int(e) for e in rng.permutation(n)[: int(rng.integers(0, n))])
        budget = int(rng.integers(0, 10))
        slots = int(rng.integers(1, 12))
        ranking = sorted(range(n), key=lambda e: (-s[e], e))
        got, last = P.select_prefetch(ranking, lambda e: e in resident, budget, slots)
        # brute force: sort everything, filter, truncate
        want = [e for e in ranking if e not in resident][: min(budget, slots)]
        assert got == want
        assert len(got) <= budget and not (set(got) & resident)
        assert all((-s[a], a) < (-s[b], b) for a, b in zip(got, got[1:]))   # descending priority
        assert (last == -1) if not got else ranking[last] == got[-1]


# ---------------------------------------------------------------- LRU against OrderedDict
def test_demand_matches_ordereddict_lru():
    # one expert per demand: ticks are all distinct, so the policy is textbook LRU
    n, S = 12, 4
    tbl = P.SlotPolicy(1, n, S)
    lru = OrderedDict()
    for _ in range(500):
        e = int(rng.integers(0, n))
        waves = tbl.demand(0, [e])
        hit = e in lru
        if hit:
            lru.move_to_end(e)
        else:
            if len(lru) == S:
                lru.popitem(last=False)
            lru[e] = True
        assert waves[0][0][2] == (not hit)
        assert tbl.resident(0) == sorted(lru)


def test_cyclic_trace_closed_forms():
    n, S, K = 16, 8, 2
    # working set fits: 100 % hits after the first lap
    tbl = P.SlotPolicy(1, n, S)
    cyc = [[0, 1], [2, 3], [4, 5], [6, 7]]
    for lap in range(5):
        for need in cyc:
            tbl.demand(0, need)
    assert tbl.stats.misses == 8 and tbl.stats.hits == 4 * 4 * K
    # working set one too large, visited in LRU order: 0 % hits forever
    tbl = P.SlotPolicy(1, n, S)
    cyc = [[0, 1], [2, 3], [4, 5], [6, 7], [8, 9]]
    for lap in range(5):
        for need in cyc:
            tbl.demand(0, need)
    assert tbl.stats.hits == 0 and tbl.stats.misses == 5 * 5 * K


def test_empty_slots_first_then_lowest_tick_then_lowest_id():
    tbl = P.SlotPolicy(1, 10, 3)
    assert [w[1] for w in tbl.demand(0, [7, 5])[0]] == [0, 1]     # ascending id into slots 0,1
    assert tbl.pools[0].slot_expert == [5, 7, -1]
    tbl.demand(0, [9])                                            # empty slot 2
    assert tbl.pools[0].slot_expert == [5, 7, 9]
    tbl.demand(0, [1])                                            # 5 and 7 share the oldest tick: lower id goes
    assert tbl.pools[0].slot_expert == [1, 7, 9]
    ev = [e for e in tbl.events if e[2] == "EVICT"]
    assert ev == [(0, 0, "EVICT", 5, 0)]


def test_waves_when_demand_exceeds_slots():
    tbl = P.SlotPolicy(1, 20, 4)
    waves = tbl.demand(0, range(10))
    assert [len(w) for w in waves] == [4, 4, 2]
    assert [e for w in waves for e, _, _ in w] == list(range(10))
    assert tbl.stats.waves == 2 and tbl.stats.misses == 10
    # second call: the survivors of the last wave hit, and hits sit in wave 0
    waves = tbl.demand(0, range(10))
    hits = [e for e, _, m in waves[0] if not m]
    assert hits == [6, 7, 8, 9]      # wave 3 (8, 9) evicted the two lowest ids of wave 2 (4, 5)
    # slot table stays a bijection
    check_bijection(tbl, 0)


def check_bijection(tbl, l):
    pool = tbl.pools[l]
    for s, e in enumerate(pool.slot_expert):
        if e >= 0:
            assert pool.expert_slot[e] == s
    for e, s in enumerate(pool.expert_slot):
        if s >= 0:
            assert pool.slot_expert[s] == e
    occupied = [e for e in pool.slot_expert if e >= 0]
    assert len(occupied) == len(set(occupied))


# ---------------------------------------------------------------- prefetch
def test_prefetch_excludes_resident_and_respects_budget():
    n, S = 16, 6
    tbl = P.SlotPolicy(2, n, S)
    tbl.demand(1, [3, 4])
    ranking = [4, 9, 3, 1, 12, 0] + [e for e in range(n) if e not in (4, 9, 3, 1, 12, 0)]
    sel, protect = tbl.plan(1, ranking, 3)
    assert sel == [9, 1, 12]                   # 4 and 3 are resident
    assert protect == [4, 3]                   # both outrank the last selected (12)
    issued = tbl.prefetch(1, sel, protect)
    assert [e for e, _ in issued] == [9, 1, 12]
    # a second request at the same priorities issues nothing twice (A ∪ U excluded)
    sel2, _ = tbl.plan(1, ranking, 3)
    assert not set(sel2) & {9, 1, 12, 3, 4}
    check_bijection(tbl, 1)


def test_predicted_use_touch_protects_ranked_residents():
    n, S = 8, 3
    tbl = P.SlotPolicy(2, n, S)
    tbl.demand(1, [0]); tbl.demand(1, [1]); tbl.demand(1, [2])     # LRU order 0,1,2
    ranking = [0, 5, 6, 7, 1, 2, 3, 4]        # resident 0 is predicted most needed
    sel, protect = tbl.plan(1, ranking, 1)
    assert sel == [5] and protect == [0]
    tbl.prefetch(1, sel, protect)
    assert tbl.resident(1) == [0, 2, 5]       # victim was 1, not the older-but-predicted 0
    plain = P.SlotPolicy(2, n, S, plain_lru=True)
    plain.demand(1, [0]); plain.demand(1, [1]); plain.demand(1, [2])
    sel, protect = plain.plan(1, ranking, 1)
    plain.prefetch(1, sel, protect)
    assert plain.resident(1) == [1, 2, 5]     # literal LRU evicts the predicted expert


def test_prefetch_never_evicts_same_batch_and_stops_when_full():
    n, S = 10, 3
    tbl = P.SlotPolicy(2, n, S)
    tbl.demand(1, [0, 1, 2])
    ranking = [0, 1, 9, 8, 7] + [2, 3, 4, 5, 6]
    sel, protect = tbl.plan(1, ranking, 3)
    assert sel == [9, 8, 7] and protect == [0, 1]
    issued = tbl.prefetch(1, sel, protect)
    assert [e for e, _ in issued] == [9]       # only one unprotected slot exists
    assert tbl.resident(1) == [0, 1, 9]


def test_wasted_and_first_use_accounting():
    tbl = P.SlotPolicy(2, 8, 2)
    tbl.prefetch(1, [5, 6], [])
    tbl.demand(1, [5])
    assert tbl.events[-1] == (0, 1, "HIT_PREFETCHED", 5, 0)
    tbl.demand(1, [5])
    assert tbl.events[-1][2] == "HIT"
    tbl.demand(1, [7])                          # evicts 6, prefetched and never used
    kinds = [e[2] for e in tbl.events]
    assert "EVICT_WASTED" in kinds and tbl.stats.wasted == 1 and tbl.stats.hits_prefetched == 1


# ---------------------------------------------------------------- on-demand vs perfect knowledge
@pytest.mark.parametrize("budget", [1, 2, 4, 8])
def test_hint_trace_equals_on_demand_in_copies_and_residency(budget):
    L, n, S, K, steps = 4, 32, 8, 4, 120
    r = np.random.default_rng(5)
    trace = [[sorted(int(e) for e in r.permutation(n)[:K]) for _ in range(L)] for _ in range(steps)]
    od = P.SlotPolicy(L, n, S)
    pk = P.SlotPolicy(L, n, S)
    for t in range(steps):
        for l in range(L):
            od.demand(l, trace[t][l])
            pk.demand(l, trace[t][l])
            assert od.resident(l) == pk.resident(l)          # same resident SET after every demand
            if l <= L - 2:
                sel, protect = pk.plan(l + 1, trace[t][l + 1], budget, protect_all=True)
                assert len(sel) <= budget
                pk.prefetch(l + 1, sel, protect)
        od.step += 1; pk.step += 1
    assert od.stats.misses == pk.stats.misses + pk.stats.prefetch_issued   # same number of copies
    assert pk.stats.wasted == 0
    if budget >= K:
        # every layer >= 1 is fully covered: its demand phase never misses
        late = [e for e in pk.events if e[2] == "MISS" and e[1] >= 1]
        assert late == []


def test_pred0_changes_nothing():
    L, n, S = 2, 8, 3
    a = P.SlotPolicy(L, n, S); b = P.SlotPolicy(L, n, S)
    for need in ([1, 2], [3], [1, 4]):
        a.demand(1, need); b.demand(1, need)
        sel, _ = b.plan(1, list(range(n)), 2)
        b.plan_only(1, sel)
        assert a.pools[1].slot_expert == b.pools[1].slot_expert
    assert b.stats.planned > 0 and b.stats.prefetch_issued == 0
