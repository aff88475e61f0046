"""Closed-form adapter stand-ins (truncated SVD of the next gate, reduced-rank regression): the
host-side math against textbook identities, and on the GPU the adapters they produce run through
the library with the oracle's decisions."""
import numpy as np
import pytest
import torch

import synth
from paper_2607_24787_b200.adapter_fit import reduced_rank_fit, svd_adapter


def test_svd_adapter_is_best_low_rank_approximation():
    g = torch.Generator().manual_seed(0)
    w = torch.randn(12, 40, generator=g)
    s = torch.linalg.svdvals(w.double())
    for r in (1, 5, 12):
        a, b = svd_adapter(w, r)
        assert a.shape == (r, 40) and b.shape == (12, r)
        err = torch.linalg.norm(w.double() - b.double() @ a.double())
        assert abs(err - s[r:].pow(2).sum().sqrt()) < 1e-5       # Eckart-Young
    a, b = svd_adapter(w, 16)                                      # rank above min(n, D): zero padding
    assert a.shape == (16, 40) and torch.allclose(b @ a, w, atol=1e-5)


def test_reduced_rank_fit_recovers_an_exactly_low_rank_map():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(200, 24, generator=g)
    c0 = torch.randn(24, 3, generator=g) @ torch.randn(3, 10, generator=g)
    a, b = reduced_rank_fit(x, x @ c0, rank=3, ridge=1e-12)
    assert torch.allclose(a.T @ b.T, c0, atol=1e-4)


def test_reduced_rank_fit_error_decomposition():
    # ||z - x C_r||^2 = ||z - x C_ols||^2 + sum of the discarded squared singular values of x C_ols
    g = torch.Generator().manual_seed(2)
    x = torch.randn(300, 20, generator=g).double()
    z = (x @ torch.randn(20, 9, generator=g).double()) + 0.3 * torch.randn(300, 9, generator=g).double()
    c_ols = torch.linalg.lstsq(x, z).solution
    sv = torch.linalg.svdvals(x @ c_ols)
    base = (z - x @ c_ols).pow(2).sum()
    for r in (1, 4, 9):
        a, b = reduced_rank_fit(x, z, rank=r, ridge=1e-13)
        err = (z - x @ (a.double().T @ b.double().T)).pow(2).sum()
        want = base + sv[r:].pow(2).sum()
        assert abs(err - want) / want < 2e-3            # the factors come back in fp32


def test_reduced_rank_fit_underdetermined_interpolates():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(16, 64, generator=g)           # fewer samples than inputs
    z = torch.randn(16, 8, generator=g)
    a, b = reduced_rank_fit(x, z, rank=8, ridge=1e-10)
    assert torch.allclose(x @ a.T @ b.T, z, atol=1e-3)


def _build(cfg, **kw):
    from paper_2607_24787_b200.build import build as b
    from paper_2607_24787_b200.synth_model import build_from_synth
    b()
    return build_from_synth(cfg, **kw)


def _rows(cfg, steps, stream=0):
    tok = synth.zipf_tokens(cfg, steps=steps, stream=stream)
    return synth.embedding_rows(cfg, tok.reshape(-1)).view(steps, cfg.batch, cfg.hidden).contiguous()


@pytest.mark.gpu
def test_full_rank_svd_adapter_ranks_like_gate_reuse():
    cfg = synth.get_config("tiny")
    H = _rows(cfg, 4).cuda()
    orders = []
    for kind in ("gate_reuse", "svd"):
        m = _build(synth.get_config("tiny", adapter_rank=cfg.n_experts), adapter=kind)
        got = []
        for s in range(4):
            x, ids, w, _ = m.router_topk(0, H[s])
            m.synchronize()
            scores, order = m.adapter_predict(0, x)
            got.append((scores.copy(), order.copy()))
        orders.append(got)
        m.close()
    for (s0, o0), (s1, o1) in zip(*orders):
        assert np.allclose(s0, s1, atol=2e-4)
        assert o0[0] == o1[0]


@pytest.mark.gpu
def test_fitted_adapter_predicts_its_calibration_stream_and_keeps_outputs():
    from paper_2607_24787_b200.synth_model import collect_router_io, fitted_adapters
    from helpers import SynthWeights, make_ref, f64
    from oracle import ref_math as M
    cfg = synth.get_config("tiny", adapter_rank=16, budget=2)
    steps = 48
    H = _rows(cfg, steps, stream=5)
    m = _build(cfg)
    X, Z = collect_router_io(m, H.cuda())
    m.set_policy("adapter"); m.cache_reset(); m.reset_stats()
    for s in range(steps):
        m.decode_step(H[s].cuda())
    m.synchronize()
    st = m.stats()
    chance = st["recall_sum"] / st["recall_count"]
    m.close()
    a, b = fitted_adapters(X, Z, cfg.adapter_rank, torch.float32)
    m = _build(cfg, adapter=(a, b))

    class W(SynthWeights):                     # the oracle sees the same fitted adapters
        def adapter(self, l):
            return f64(a[l]), f64(b[l])

    ref = make_ref(cfg, weights=W(cfg), policy="adapter")
    m.set_policy("adapter")
    for s in range(steps):
        out = m.decode_step(H[s].cuda())
        m.synchronize()
        want, _ = ref.step(H[s].numpy())
        assert M.rel_linf(out.cpu().numpy().astype(np.float64)[0], want[0]) < 4e-5
    assert m.events() == ref.table.events
    st = m.stats()
    fitted = st["recall_sum"] / st["recall_count"]
    m.close()
    # rank n with fewer samples than inputs interpolates the calibration stream
    assert fitted > 0.9 and chance < 0.5, (fitted, chance)
