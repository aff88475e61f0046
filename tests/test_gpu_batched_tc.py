"""Batched decode on the tensor-core path (grouped tcgen05 FFN): parity with the CPU oracle.

The tensor cores take bf16 activations, so outputs are held to the bf16 tolerance 2e-2
(max|a-b| / max|b| per row). Because a 1e-3 perturbation of the hidden state can flip a Top-K
choice far from a 1e-5 near-tie, whole-step parity is teacher-forced per layer: every layer gets
the oracle's input, its expert ids must match bit-exactly (near-ties excepted) and its output must
agree within tolerance. Cache events of a free-running run are checked against the policy oracle
replayed on the GPU's own demand sets.
"""
import numpy as np
import pytest
import torch

import synth
from helpers import SynthWeights, make_ref
from oracle import ref_math as M, ref_policy as P

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2

CASES = {
    # (config, batch): several j-tiles and d-tiles, more distinct experts than slots -> waves
    "small_waves": (synth.get_config("qwen3", n_layers=2, hidden=256, n_experts=24, inter=256, top_k=4, slots=6, budget=2), 17),
    "wide": (synth.get_config("qwen3", n_layers=2, hidden=1280, n_experts=16, inter=384, top_k=3, slots=16, budget=2), 64),
    "one_wave_many_tokens": (synth.get_config("qwen3", n_layers=3, hidden=512, n_experts=8, inter=128, top_k=2, slots=8, budget=1), 64),
    # the largest top-k the boundary allows minus shared experts: the combine kernel's block is 32 x K threads
    "many_k": (synth.get_config("qwen3", n_layers=2, hidden=256, n_experts=32, inter=256, top_k=16, slots=32, budget=2), 9),
    # 4-bit experts de-quantised inside the grouped kernel (scales every fourth K-block / second d-tile)
    "q4_small_waves": (synth.get_config("qwen3_q4", n_layers=2, hidden=256, n_experts=24, inter=256, top_k=4, slots=6, budget=2), 17),
    "q4_wide": (synth.get_config("qwen3_q4", n_layers=2, hidden=1280, n_experts=16, inter=384, top_k=3, slots=16, budget=2), 64),
    "q4_deep": (synth.get_config("qwen3_q4", n_layers=2, hidden=2048, n_experts=8, inter=128, top_k=2, slots=8, budget=1), 33),
}


def dev(a):
    t = torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float32).cuda()
    torch.cuda.synchronize()
    return t


@pytest.fixture(scope="module", params=list(CASES))
def setup(request):
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.synth_model import build_from_synth
    build()
    cfg, nb = CASES[request.param]
    cfg = cfg.replace(batch=nb)
    m = build_from_synth(cfg)
    wts = SynthWeights(cfg)
    steps = 3
    tok = synth.zipf_tokens(cfg, steps=steps)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(steps, nb, cfg.hidden)
    yield cfg, nb, m, wts, H
    m.close()


def test_teacher_forced_layers(setup):
    cfg, nb, m, wts, H = setup
    m.cache_reset()
    ref = make_ref(cfg, weights=wts, budget=2, policy=P.ON_DEMAND)
    flagged = 0
    for s in range(H.shape[0]):
        _, recs = ref.step(H[s])
        h_in = H[s].astype(np.float64)
        for l, rec in enumerate(recs):
            hd = dev(h_in)
            x, ids, w, _ = m.router_topk(l, hd)
            tie = [M.near_tie(rec.logits[t], cfg.top_k) for t in range(nb)]
            for t in range(nb):
                if tie[t]:
                    flagged += 1
                else:
                    assert list(ids[t]) == list(rec.ids[t]), (s, l, t)
            m.moe_ffn(l, x, ids, w, hd)
            m.synchronize()
            got = hd.cpu().numpy().astype(np.float64)
            for t in range(nb):
                if not tie[t]:
                    assert M.rel_linf(got[t] - h_in[t], rec.h_out[t] - h_in[t]) < TOL_BF16, (s, l, t)
                    assert M.rel_linf(got[t], rec.h_out[t]) < TOL_BF16
            h_in = rec.h_out                      # teacher forcing: next layer starts from the oracle's state
    assert flagged < 0.01 * H.shape[0] * cfg.n_layers * nb + 1
    st = m.stats()
    assert st["ffn_launches"] > 0


def test_tensor_core_path_agrees_with_gemv_path(setup):
    cfg, nb, m, wts, H = setup
    outs = {}
    for mode in (0, 1):
        m.cache_reset()
        m.set_batched_path(mode)
        m.set_policy("on_demand")
        hd = dev(H[0])
        x, ids, w, _ = m.router_topk(0, hd)
        m.moe_ffn(0, x, ids, w, hd)
        m.synchronize()
        outs[mode] = hd.cpu().numpy().astype(np.float64) - H[0]
    m.set_batched_path(0)
    for t in range(nb):
        assert M.rel_linf(outs[0][t], outs[1][t]) < TOL_BF16
    assert not np.array_equal(outs[0], outs[1])            # really two different kernels (bf16 vs fp32 activations)


def test_free_running_events_match_policy_oracle(setup):
    cfg, nb, m, wts, H = setup
    m.cache_reset()
    m.set_policy("on_demand")
    for s in range(H.shape[0]):
        out = m.decode_step(dev(H[s]))
    m.synchronize()
    assert np.all(np.isfinite(out.cpu().numpy()))
    ev = m.events()
    # demand sets as the GPU routed them, then the policy oracle on exactly those sets
    need = {}
    for (s, l, kind, e, slot) in ev:
        if kind in ("HIT", "HIT_PREFETCHED", "MISS"):
            need.setdefault((s, l), []).append(e)
    ref = P.SlotPolicy(cfg.n_layers, cfg.n_experts, cfg.slots)
    for s in range(H.shape[0]):
        for l in range(cfg.n_layers):
            ref.demand(l, need[(s, l)])
        ref.step += 1
    assert ev == ref.events
    if cfg.slots < cfg.n_experts and nb * cfg.top_k > cfg.slots:
        assert m.stats()["waves"] > 0


def test_offloaded_waves_give_the_bits_of_a_fully_resident_context(setup):
    """Router-preserving guarantee for batched decode (Section 3.1, last paragraph; Section 3.3, last
    paragraph), bit for bit: a (token, expert) pair's partial output does not depend on the wave its
    expert is computed in, and one combine per layer adds a token's experts in rank order, so a
    context with fewer slots than experts (waves, on-demand loads, prefetches, evictions) and a
    context that holds every expert (host-free steps, plan built on the device) agree exactly."""
    from paper_2607_24787_b200.synth_model import build_from_synth
    cfg, nb, m, wts, H = setup
    outs = {}
    for policy in ("adapter", "on_demand"):
        m.cache_reset(); m.set_policy(policy); m.set_budget(2)
        o = [m.decode_step(dev(H[s])) for s in range(H.shape[0])]
        m.synchronize()
        outs[policy] = np.stack([x.cpu().numpy() for x in o])
    assert np.array_equal(outs["adapter"], outs["on_demand"])
    full = build_from_synth(cfg, slots=cfg.n_experts, budget=0)
    try:
        full.set_policy("on_demand")
        o = [full.decode_step(dev(H[s])) for s in range(H.shape[0])]
        full.synchronize()
        got = np.stack([x.cpu().numpy() for x in o])
        assert full.stats()["misses"] > 0          # the first step loads; later steps run without a host turn
        assert np.array_equal(got, outs["on_demand"])
    finally:
        full.close()


def test_device_side_wait_in_the_producer_warp_is_bit_identical(setup):
    """The grouped kernels' producer warp can wait for a unit's expert copy itself (per unit, on the
    batch's arrival counter) instead of the host ordering the launch behind the copy events: same
    outputs, same cache events, and some launches really had copies in flight."""
    from paper_2607_24787_b200 import binding as B
    cfg, nb, m, wts, H = setup
    runs = {}
    for on in (0, 1):
        m.cache_reset(); m.set_policy("adapter"); m.set_budget(2)
        try:
            m.set_device_wait(on)
        except B.SpmError:
            pytest.skip("stream-ordered memory writes are not available on this driver")
        outs = []
        for s in range(H.shape[0]):
            outs.append(m.decode_step(dev(H[s])))
        m.synchronize()
        runs[on] = (np.stack([o.cpu().numpy() for o in outs]), m.events(), m.stats())
    m.set_device_wait(0)
    assert np.array_equal(runs[0][0], runs[1][0]) and runs[0][1] == runs[1][1]
    assert runs[1][2]["misses"] > 0 and runs[1][2]["ffn_launches"] > 0
    m.check_invariants()


@pytest.mark.parametrize("name", ["small_waves", "q4_small_waves"])
def test_producer_warp_wait_runs_out_and_the_context_survives(name):
    """An arrival counter that is never bumped (withheld on the host; the bytes land) makes the
    producer warp's wait run out after the configured limit: the kernel winds down, the host reads
    SPM_ERR_TIMEOUT once, and after a cache reset the same context computes the same outputs as a
    context that never waited on the device."""
    import time
    from paper_2607_24787_b200 import binding as B
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.synth_model import build_from_synth
    build()
    cfg, nb = CASES[name]
    cfg = cfg.replace(batch=nb)
    tok = synth.zipf_tokens(cfg, steps=2)
    H = synth.embedding_rows(cfg, tok.reshape(-1)).numpy().reshape(2, nb, cfg.hidden)
    m = build_from_synth(cfg)
    try:
        m.set_policy("on_demand")
        want = []
        for s in range(2):
            want.append(m.decode_step(dev(H[s])))
        m.synchronize()
        want = [o.cpu().numpy() for o in want]
        try:
            m.set_device_wait(1)
        except B.SpmError:
            pytest.skip("stream-ordered memory writes are not available on this driver")
        m.set_device_wait_limit_us(3000)
        m.cache_reset()
        m.test_withhold_arrivals(1)
        t0 = time.perf_counter()
        with pytest.raises(B.SpmError) as e:
            m.decode_step(dev(H[0]))
            m.synchronize()
        assert e.value.code == -4                    # SPM_ERR_TIMEOUT
        assert time.perf_counter() - t0 < 1.9        # the configured limit applied, not the 2 s default
        m.synchronize()                              # reported once
        m.set_device_wait_limit_us(0)
        m.cache_reset()
        for s in range(2):
            out = m.decode_step(dev(H[s]))
            m.synchronize()
            assert np.array_equal(out.cpu().numpy(), want[s])
        m.check_invariants()
    finally:
        m.close()


WIDTH_CASES = {
    "bf16": synth.get_config("qwen3", n_layers=1, hidden=512, n_experts=8, inter=256, top_k=3, slots=8, budget=1),
    "q4": synth.get_config("qwen3_q4", n_layers=1, hidden=512, n_experts=8, inter=256, top_k=3, slots=8, budget=1),
}


@pytest.mark.parametrize("name", list(WIDTH_CASES))
def test_every_tokens_per_expert_width(name):
    """The grouped kernel issues its MMAs with N = the unit's tokens rounded up to 16 and fetches
    16, 32 or 64 token rows: experts with 64, 47, 33, 17, 16, 14 and 1 tokens in one launch, each
    token's output against the oracle's dense definition."""
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.synth_model import build_from_synth
    build()
    nb = 64
    cfg = WIDTH_CASES[name].replace(batch=nb)
    m = build_from_synth(cfg)
    try:
        wts = SynthWeights(cfg)
        ids = np.zeros((nb, 3), dtype=np.int32)                     # expert 0: all 64 tokens
        ids[:, 1] = np.where(np.arange(nb) < 47, 1, 2)              # expert 1: 47 tokens, expert 2: 17
        third = np.full(nb, 6, dtype=np.int32)                      # expert 6: 14 tokens
        third[:33] = 3                                              # expert 3: 33
        third[33:49] = 4                                            # expert 4: 16
        third[49] = 5                                               # expert 5: 1
        ids[:, 2] = third
        counts = np.bincount(ids.reshape(-1), minlength=8)
        assert sorted(counts.tolist(), reverse=True)[:7] == [64, 47, 33, 17, 16, 14, 1]
        rng = np.random.default_rng(11)
        x = rng.standard_normal((nb, cfg.hidden)).astype(np.float32)
        w = rng.uniform(0.1, 1.0, size=(nb, 3)).astype(np.float32)
        w /= w.sum(axis=1, keepdims=True)
        xd, wd = dev(x), dev(w)
        hd = torch.zeros(nb, cfg.hidden, device="cuda")
        m.moe_ffn(0, xd, ids, wd, hd)
        m.synchronize()
        got = hd.cpu().numpy().astype(np.float64)
        experts = lambda e: wts.expert(0, e)
        for t in range(nb):
            want = M.moe_ffn(x[t].astype(np.float64), ids[t], w[t].astype(np.float64), experts)
            assert M.rel_linf(got[t], want) < TOL_BF16, (name, t)
        assert m.stats()["ffn_launches"] == 1
    finally:
        m.close()
