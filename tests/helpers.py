"""Test-side glue: feeds the synthetic inputs to the CPU oracle as float64 numpy arrays."""
from __future__ import annotations

from functools import lru_cache

import numpy as np
import torch

import synth


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


class SynthWeights:
    """The oracle's weight provider, backed by the counter-based generator."""

    def __init__(self, cfg: synth.ModelCfg, gamma=None, cache_experts=True):
        self.cfg = cfg
        self._gamma = gamma
        self._cache = {} if cache_experts else None

    def gamma(self, l):
        if self._gamma is not None:
            return np.asarray(self._gamma[l], np.float64)
        return np.ones(self.cfg.hidden)

    @lru_cache(maxsize=None)
    def router(self, l):
        return f64(synth.router_w(self.cfg, l))

    @lru_cache(maxsize=None)
    def adapter(self, l):
        return f64(synth.adapter_a(self.cfg, l)), f64(synth.adapter_b(self.cfg, l))

    def expert(self, l, e):
        if self._cache is not None and (l, e) in self._cache:
            return self._cache[(l, e)]
        g, u, d = synth.expert_matrices(self.cfg, l, [e])
        trip = (f64(g[0]), f64(u[0]), f64(d[0]))
        if self._cache is not None:
            self._cache[(l, e)] = trip
        return trip

    def shared(self, l):
        n = self.cfg.n_experts
        return [self.expert(l, n + s) for s in range(self.cfg.n_shared)]


def make_ref(cfg: synth.ModelCfg, policy="adapter", budget=None, slots=None, weights=None, **kw):
    from oracle.ref_decode import RefDecoder
    wts = weights if weights is not None else SynthWeights(cfg)
    b = cfg.budget if budget is None else budget
    return RefDecoder(cfg.n_layers, cfg.hidden, cfg.n_experts, cfg.top_k, wts,
                      cfg.slots if slots is None else slots, b, policy=policy,
                      renormalize=bool(cfg.renormalize), rms_eps=cfg.rms_eps, **kw)
