"""CPU oracle, policy part: expert slot table, demand resolution and budgeted prefetch.

TEST INFRASTRUCTURE ONLY. Pure integer / ordering logic, plain Python loops,
no code shared with the CUDA library's host runtime.

What the paper fixes (Section 3.3, "Window-Aware Prefetch Budgeting"):
  * experts already available (A) or in transfer (U) are excluded from new requests;
  * the remaining experts are ranked by predicted priority s_e and the first
    M_max are selected: P = Top_{M_max}({s_e : e not in A ∪ U});
  * they are transferred in descending priority and m = |P| <= M_max;
  * whatever the router asks for and the cache lacks at execution time is fetched
    then (the on-demand fallback), which is why a wrong prediction can cost time
    but can never change routing or outputs.
The paper does not say how the accelerator-side cache is organised. The reading
taken here: S slots per layer, least-recently-used eviction driven by one global
tick, ties broken by the lower expert id, empty slots taken lowest index first,
demand copies of a layer ordered before the prefetch copies for the next one, and
a "predicted-use touch": before a prefetch installs anything, the resident
experts that the same prediction ranks above the last selected candidate are
marked most-recently-used, so that a prefetch never evicts an expert predicted to
be needed more than what it brings in. `plain_lru=True` switches the touch off.

An expert "has a slot" from the moment a transfer into that slot is issued, so
"has a slot" is exactly membership in A ∪ U.

Pinned by tests/test_oracle_policy.py (brute-force selection, an independent
OrderedDict LRU, closed-form hit rates on cyclic traces, the on-demand /
perfect-knowledge copy-count identity, invariants).
"""
from __future__ import annotations

from dataclasses import dataclass, field

DEMAND = 0
PREFETCH = 1

# policies
ADAPTER = "adapter"          # prefetch what the adapter ranks highest
ON_DEMAND = "on_demand"      # no prediction, no prefetch (the paper's OFF arm)
HINT_TRACE = "hint_trace"    # perfect knowledge: ranking = the true next-layer experts
PRED0 = "pred0"              # predict and select, issue nothing (the paper's PRED0 arm)
NAIVE = "naive"              # prefetch what the preceding token used at that layer (the paper's Naive Prefetch arm)


@dataclass
class Pool:
    slot_expert: list
    slot_tick: list
    slot_origin: list
    slot_used: list
    expert_slot: list


@dataclass
class Stats:
    hits: int = 0
    hits_prefetched: int = 0
    misses: int = 0
    evictions: int = 0
    wasted: int = 0
    prefetch_issued: int = 0
    touches: int = 0
    waves: int = 0
    planned: int = 0


def borda_ranking(ids_per_token, n_experts: int):
    """Experts used by a batch, ranked by sum over tokens of (K - rank position), ties to the lower id.

    For one token this is the router's own rank order. Used by the Naive Prefetch arm, which
    replays the previous token's experts as the prediction (Section 4.4, Table 5)."""
    score = [0] * n_experts
    for ids in ids_per_token:
        K = len(ids)
        for pos, e in enumerate(ids):
            score[int(e)] += K - pos
    used = [e for e in range(n_experts) if score[e] > 0]
    return sorted(used, key=lambda e: (-score[e], e))


def select_prefetch(ranking, has_slot, budget: int, slots: int):
    """P of Section 3.3: walk the ranking, skip experts in A ∪ U, keep the first `budget`.

    `ranking` lists expert ids in descending priority (all n experts for the
    adapter, only the truly needed ones for perfect knowledge). Returns (P, last)
    where last is the position in `ranking` of P's final member (-1 if P is empty).
    """
    P = []
    last = -1
    limit = min(budget, slots)
    for pos, e in enumerate(ranking):
        if len(P) >= limit:
            break
        if not has_slot(e):
            P.append(e)
            last = pos
    return P, last


class SlotPolicy:
    """Slot tables of all layers plus the event log."""

    def __init__(self, n_layers: int, n_experts: int, slots: int, plain_lru: bool = False):
        if slots < 1:
            raise ValueError("need at least one slot")
        self.L, self.n, self.S = n_layers, n_experts, slots
        self.plain_lru = plain_lru
        self.reset()

    def reset(self):
        self.tick = 0
        self.step = 0
        self.pools = [Pool([-1] * self.S, [0] * self.S, [DEMAND] * self.S, [0] * self.S,
                           [-1] * self.n) for _ in range(self.L)]
        self.events = []  # (step, layer, kind, expert, slot)
        self.stats = Stats()

    # ---- helpers -------------------------------------------------------
    def _log(self, layer, kind, expert, slot):
        self.events.append((self.step, layer, kind, expert, slot))

    def has_slot(self, layer, e) -> bool:
        return self.pools[layer].expert_slot[e] >= 0

    def resident(self, layer) -> list:
        return sorted(e for e in self.pools[layer].slot_expert if e >= 0)

    def _victim(self, pool):
        for s in range(self.S):
            if pool.slot_expert[s] < 0:
                return s
        best, best_key = None, None
        for s in range(self.S):
            if pool.slot_tick[s] < self.tick:
                key = (pool.slot_tick[s], pool.slot_expert[s])
                if best is None or key < best_key:
                    best, best_key = s, key
        return best

    def _install(self, layer, pool, s, e, origin):
        v = pool.slot_expert[s]
        if v >= 0:
            wasted = pool.slot_origin[s] == PREFETCH and not pool.slot_used[s]
            self._log(layer, "EVICT_WASTED" if wasted else "EVICT", v, s)
            self.stats.evictions += 1
            self.stats.wasted += int(wasted)
            pool.expert_slot[v] = -1
        pool.slot_expert[s] = e
        pool.slot_tick[s] = self.tick
        pool.slot_origin[s] = origin
        pool.slot_used[s] = 1 if origin == DEMAND else 0
        pool.expert_slot[e] = s

    # ---- demand --------------------------------------------------------
    def demand(self, layer: int, need):
        """Resolve the batch demand of `layer`.

        Returns a list of waves; each wave is a list of (expert, slot, missed).
        A new wave starts only when more distinct experts are needed than there
        are slots: the experts placed so far must be computed before their slots
        can be reused.
        """
        pool = self.pools[layer]
        need = sorted(set(int(e) for e in need))
        self.tick += 1
        waves = [[]]
        missing = []
        for e in need:
            s = pool.expert_slot[e]
            if s >= 0:
                first_use = pool.slot_origin[s] == PREFETCH and not pool.slot_used[s]
                self._log(layer, "HIT_PREFETCHED" if first_use else "HIT", e, s)
                self.stats.hits += 1
                self.stats.hits_prefetched += int(first_use)
                pool.slot_used[s] = 1
                pool.slot_tick[s] = self.tick
                waves[0].append((e, s, False))
            else:
                missing.append(e)
        for e in missing:
            s = self._victim(pool)
            if s is None:
                self._log(layer, "WAVE", len(waves), -1)
                self.stats.waves += 1
                self.tick += 1
                waves.append([])
                s = self._victim(pool)
            self._install(layer, pool, s, e, DEMAND)
            self._log(layer, "MISS", e, s)
            self.stats.misses += 1
            waves[-1].append((e, s, True))
        return waves

    # ---- prefetch ------------------------------------------------------
    def plan(self, layer: int, ranking, budget: int, protect_all: bool = False):
        """(P, protect): the selection of Section 3.3 for target pool `layer`, and the
        resident experts the predicted-use touch will protect.

        protect_all=False: residents ranked above P's last member (adapter ranking).
        protect_all=True: every resident expert in `ranking` (perfect knowledge,
        where `ranking` holds exactly the experts that will be needed).
        """
        pool = self.pools[layer]
        P, last = select_prefetch(ranking, lambda e: pool.expert_slot[e] >= 0, budget, self.S)
        if self.plain_lru:
            return P, []
        if protect_all:
            protect = [e for e in ranking if pool.expert_slot[e] >= 0]
        else:
            protect = [e for e in ranking[:max(last, 0)] if pool.expert_slot[e] >= 0] if P else []
        return P, protect

    def prefetch(self, layer: int, P, protect, dropped=()):
        """Install P into pool `layer` in the given (descending-priority) order.

        Returns the list of (expert, slot) actually issued. Stops early when every
        slot is protected. Experts in `dropped` are skipped as if the transfer
        request had been lost (fault injection): they get no slot.
        """
        pool = self.pools[layer]
        self.tick += 1
        for e in protect:
            s = pool.expert_slot[e]
            pool.slot_tick[s] = self.tick
            self._log(layer, "TOUCH_PRED", e, s)
            self.stats.touches += 1
        issued = []
        for e in P:
            if e in dropped:
                self._log(layer, "DROPPED", e, -1)
                continue
            s = self._victim(pool)
            if s is None:
                break
            self._install(layer, pool, s, e, PREFETCH)
            self._log(layer, "PREFETCH", e, s)
            self.stats.prefetch_issued += 1
            issued.append((e, s))
        return issued

    def plan_only(self, layer: int, P):
        """PRED0: record the selection, touch nothing."""
        for e in P:
            self._log(layer, "PLAN", e, -1)
            self.stats.planned += 1
