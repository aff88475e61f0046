"""CPU oracle: the whole offloaded-MoE decode step, layer by layer.

TEST INFRASTRUCTURE ONLY (tests, the smoke check and the benchmark's CPU
baseline). It composes oracle/ref_math.py (the plain layer definition, fp64) and
oracle/ref_policy.py (slot table + budgeted prefetch) in the order of the paper's
timeline (Section 3.1 and 3.3, Figure 2): at layer l the native router decides,
missing experts are loaded on demand, the adapter scores layer l+1, at most
M_max non-resident experts are requested in descending priority, the experts of
layer l run, and the residual is added.

The expert FFN reads its weights THROUGH the software slot pool (a dict
slot -> (expert id, matrices) that only MISS and PREFETCH installs write), and
asserts that the slot holds the expert the router asked for. This makes the
router-preserving guarantee (Section 3.1, last paragraph; Section 3.3, last
paragraph) a checkable property of the oracle instead of a tautology.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import ref_math as M
from . import ref_policy as P


@dataclass
class LayerRecord:
    ids: np.ndarray        # [nb, K] int64, rank order
    w: np.ndarray          # [nb, K] float64
    logits: np.ndarray     # [nb, n] float64
    x: np.ndarray          # [nb, D] float64 router input
    scores: np.ndarray | None = None   # [n] priorities for layer+1 (None on the last layer)
    order: np.ndarray | None = None    # [n] ranking of scores
    prefetch: list = field(default_factory=list)   # experts selected for layer+1, priority order
    issued: list = field(default_factory=list)     # (expert, slot) actually installed
    n_waves: int = 1
    ready: float = 1.0     # logical ReadyRecall of this layer (fraction with a slot at demand time)
    h_out: np.ndarray | None = None    # [nb, D] float64 after the residual


class RefDecoder:
    """Offloaded MoE decode on the CPU.

    weights: object with
        gamma(l) -> [D]; router(l) -> [n, D]; adapter(l) -> (A[r, D], Bup[n, r]) for l <= L-2;
        expert(l, e) -> (W_gate[I, D], W_up[I, D], W_down[D, I]); shared(l) -> list of such triples.
    """

    def __init__(self, n_layers, hidden, n_experts, top_k, weights, slots, budget,
                 policy=P.ADAPTER, renormalize=True, rms_eps=1e-6, plain_lru=False,
                 keep_records=True):
        if budget < 0:
            raise ValueError("the oracle needs an explicit budget")
        self.L, self.D, self.n, self.K = n_layers, hidden, n_experts, top_k
        self.wts = weights
        self.S, self.M_max = slots, budget
        self.policy = policy
        self.renorm = bool(renormalize)
        self.eps = rms_eps
        self.table = P.SlotPolicy(n_layers, n_experts, slots, plain_lru)
        self.storage = [dict() for _ in range(n_layers)]   # slot -> (expert, triple)
        self.drop_hook = None     # callable(step, layer, expert) -> bool: lose this prefetch request
        self.keep_records = keep_records
        self.prev_rank = [[] for _ in range(n_layers)]   # Naive Prefetch: what the preceding step used per layer

    # -- transfers into the software slot pool ----------------------------
    def _copy_in(self, layer, expert, slot):
        self.storage[layer][slot] = (expert, self.wts.expert(layer, expert))

    def _slot_weights(self, layer, expert, slot):
        assert slot >= 0 and slot in self.storage[layer], \
            f"expert {expert} of layer {layer} has no loaded slot at FFN time"
        tag, triple = self.storage[layer][slot]
        assert tag == expert, f"slot {slot} of layer {layer} holds {tag}, router asked for {expert}"
        return triple

    # -- one decode step ---------------------------------------------------
    def step(self, h_in, hint=None):
        """h_in [nb, D] -> (h_out [nb, D] float64, [LayerRecord] per layer).

        hint[l] (perfect-knowledge policy only): expert ids that layer l will truly
        need at this step, in priority order.
        """
        h = np.array(h_in, dtype=np.float64, copy=True)
        nb = h.shape[0]
        recs = []
        tbl = self.table
        for l in range(self.L):
            gamma = self.wts.gamma(l)
            W_r = self.wts.router(l)
            X = np.stack([M.rmsnorm(h[t], gamma, self.eps) for t in range(nb)])
            Z = np.stack([M.router_logits(W_r, X[t]) for t in range(nb)])
            routed = [M.route(Z[t], self.K, self.renorm) for t in range(nb)]
            ids = np.stack([r[0] for r in routed])
            w = np.stack([r[1] for r in routed])
            rec = LayerRecord(ids=ids, w=w, logits=Z, x=X)
            this_rank = P.borda_ranking(ids, self.n)

            # demand of this layer (Section 3.1, second equation) and on-demand loads
            need = M.batch_demand(ids)
            rec.ready = M.ready_recall(ids, [e for e in need if tbl.has_slot(l, e)], self.K)
            waves = tbl.demand(l, need)
            rec.n_waves = len(waves)

            # prediction for layer l+1 (Section 3.2) and budgeted prefetch (Section 3.3)
            if l <= self.L - 2:
                A, Bup = self.wts.adapter(l)
                rec.scores = M.adapter_scores(A, Bup, X)
                rec.order = M.rank_desc(M.decision_logits(rec.scores))
                if self.policy != P.ON_DEMAND:
                    if self.policy == P.HINT_TRACE:
                        ranking = [int(e) for e in hint[l + 1]]
                        sel, protect = tbl.plan(l + 1, ranking, self.M_max, protect_all=True)
                    elif self.policy == P.NAIVE:
                        sel, protect = tbl.plan(l + 1, self.prev_rank[l + 1], self.M_max)
                    else:
                        ranking = [int(e) for e in rec.order]
                        sel, protect = tbl.plan(l + 1, ranking, self.M_max)
                    rec.prefetch = list(sel)
                    if self.policy == P.PRED0:
                        tbl.plan_only(l + 1, sel)
                    else:
                        dropped = set()
                        if self.drop_hook is not None:
                            dropped = {e for e in sel if self.drop_hook(tbl.step, l + 1, e)}
                        # within one step pool l+1 is not read between now and its own
                        # demand phase, so the copies can land at once
                        rec.issued = tbl.prefetch(l + 1, sel, protect, dropped)
                        for e, s in rec.issued:
                            self._copy_in(l + 1, e, s)

            # expert computation, wave by wave (a slot is overwritten only after the
            # wave that used it has been computed)
            shared = self.wts.shared(l)
            y = np.zeros_like(h)
            for wi, wave in enumerate(waves):
                for e, s, missed in wave:
                    if missed:
                        self._copy_in(l, e, s)
                in_wave = {e: s for e, s, _ in wave}
                for t in range(nb):
                    sel_k = [k for k in range(self.K) if int(ids[t, k]) in in_wave]
                    if sel_k:
                        y[t] += M.moe_ffn(X[t], ids[t, sel_k], w[t, sel_k],
                                          lambda e: self._slot_weights(l, e, in_wave[e]))
            for t in range(nb):
                for trip in shared:
                    y[t] += M.swiglu_expert(*trip, X[t])
            h = h + y
            self.prev_rank[l] = this_rank          # becomes "the preceding token" for the next step
            rec.h_out = h.copy()
            if self.keep_records:
                recs.append(rec)
        tbl.step += 1
        return h, recs


def true_demand_trace(recs_per_step):
    """hint[step][layer]: the experts layer `layer` truly needs, ranked by true routing mass.

    Priority = sum over tokens of the renormalised routing weight (descending, ties to
    the lower id); for one token this is the router's own rank order.
    """
    out = []
    for recs in recs_per_step:
        per_layer = []
        for rec in recs:
            n = rec.logits.shape[1]
            mass = np.zeros(n)
            for t in range(rec.ids.shape[0]):
                for k in range(rec.ids.shape[1]):
                    mass[int(rec.ids[t, k])] += rec.w[t, k]
            order = [int(e) for e in M.rank_desc(mass) if mass[int(e)] > 0]
            per_layer.append(order)
        out.append(per_layer)
    return out
