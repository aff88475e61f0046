"""CPU-only checks of the C-ABI library: it builds for sm_100a, loads without a GPU, exports every
symbol include/spm.h declares, and its host-side slot table matches the policy oracle bit for bit."""
import os
import re

import numpy as np
import pytest

from oracle import ref_policy as P
from paper_2607_24787_b200 import binding as B
from paper_2607_24787_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def lib():
    build()
    return B.load()


def test_header_symbols_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "spm.h")).read()
    declared = sorted(set(re.findall(r"\b(spm_[a-z0-9_]+)\s*\(", hdr)))
    assert declared == B.EXPORTS, set(declared) ^ set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_query_and_config_errors():
    cfg = B.make_cfg(48, 2048, 128, 768, 8, 0, 16, B.DTYPE_BF16)
    assert B.spm_expert_blob_bytes(cfg) == 9437184
    assert B.spm_query_arena(cfg, 16) > 48 * 16 * 9437184
    assert B.spm_expert_blob_bytes(B.make_cfg(12, 1280, 64, 896, 6, 2, 16, B.DTYPE_Q4)) == 1935360
    with pytest.raises(B.SpmError) as e:
        B.spm_query_arena(cfg, 4)                       # slots < top_k at batch 1
    assert e.value.code == -2
    with pytest.raises(B.SpmError):
        B.spm_query_arena(B.make_cfg(2, 1000, 16, 128, 2, 0, 8, B.DTYPE_BF16), 4)   # hidden not a multiple of 256
    with pytest.raises(B.SpmError):
        B.spm_query_arena(B.make_cfg(2, 256, 16, 128, 2, 15, 8, B.DTYPE_FP32), 4)   # top_k + shared too large


def test_init_fails_loudly_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a GPU")
    cfg = B.make_cfg(2, 256, 16, 128, 2, 0, 8, B.DTYPE_FP32)
    buf = B.Buffers(256, 256, 256, 256, None, 256, 256, 1 << 40, 1, 2, 0)
    with pytest.raises(B.SpmError) as e:
        B.spm_init(cfg, 4, 2, buf)
    assert e.value.code == -3


@pytest.mark.parametrize("n_units,n_dt,grid", [(192, 16, 148), (6, 2, 148), (755, 16, 148), (148, 16, 148), (48, 10, 148),
                                              (1, 4, 7), (300, 3, 16), (40, 1, 148)])
def test_grouped_kernel_chunk_plan(n_units, n_dt, grid):
    """Phase-2 chunk list of the batched tensor-core kernel: every (unit, d-tile) exactly once, in
    unit order (the units whose phase 1 ends first come first), chunk sizes shrinking towards the
    end of the list but never below the minimum while a unit has that many d-tiles left, so that
    the CTAs that take them in order run out of work together."""
    ch = B.spm_plan_grouped_chunks(n_units, n_dt, grid)
    seen = np.zeros((n_units, n_dt), int)
    for u, dt0, dt1 in ch:
        assert 0 <= dt0 < dt1 <= n_dt
        seen[u, dt0:dt1] += 1
    assert np.all(seen == 1)
    order = [(int(u), int(d0)) for u, d0, _ in ch]
    assert order == sorted(order)
    sizes = np.array([int(d1 - d0) for _, d0, d1 in ch])
    min_chunk = min(4, n_dt)
    assert sizes.min() >= min_chunk and sizes.max() <= n_dt
    total = n_units * n_dt
    # guided: no chunk is larger than its fair share of what was left when it was cut (or the minimum, or a unit's rest)
    left = total
    for (u, d0, d1), sz in zip(ch, sizes):
        fair = -(-left // (2 * grid))
        assert sz <= max(fair, min_chunk) + min_chunk - 1, (u, d0, d1, left)
        left -= sz
    # the tail is fine-grained: the last grid chunks are all near the minimum size (when there is that much work)
    if total >= 8 * grid * min_chunk and n_dt >= 2 * min_chunk:
        assert np.all(sizes[-grid:] <= 2 * min_chunk - 1)


def test_noalloc_argument_checks_run_before_any_gpu_work():
    """The allocation-free entry point refuses bad shapes, indices and misaligned pointers on the
    host, before it touches the device: so this runs without a GPU (addresses below are never
    dereferenced)."""
    cfg = B.make_cfg(1, 2048, 8, 64, 2, 0, 4, B.DTYPE_BF16)
    ok = 1 << 20                                            # a 16-byte aligned made-up address
    for args in ((ok + 8, ok, ok, ok), (ok, ok + 2, ok, ok), (ok, ok, ok + 4, ok), (ok, ok, ok, ok + 12)):
        blobs, w, x, h = args
        with pytest.raises(B.SpmError) as e:
            B.spm_ffn_noalloc(cfg, blobs, 8, [0, 1], w, x, h)
        assert e.value.code == -1 and "aligned" in str(e.value), args
    with pytest.raises(B.SpmError) as e:
        B.spm_ffn_noalloc(B.make_cfg(1, 4096, 8, 64, 2, 0, 4, B.DTYPE_BF16), ok, 8, [0, 1], ok, ok, ok)
    assert e.value.code == -2 and "scratch" in str(e.value)
    with pytest.raises(B.SpmError) as e:
        B.spm_ffn_noalloc(cfg, ok, 8, [0, 8], ok, ok, ok)   # blob index outside the 8 blobs
    assert e.value.code == -1
    with pytest.raises(B.SpmError) as e:
        B.spm_ffn_noalloc(cfg, ok, 8, list(range(17)), ok, ok, ok)   # more experts than SPM_MAX_TOPK
    assert e.value.code == -1


def drive(policy_obj, trace, ranks, L, budget, mode, drop=0):
    """Feed one recorded trace to either the oracle SlotPolicy or the library's Sim."""
    for t, per_layer in enumerate(trace):
        for l in range(L):
            policy_obj.demand(l, per_layer[l])
            if l <= L - 2 and mode != "on_demand":
                if mode == "hint":
                    sel, prot = policy_obj.plan(l + 1, per_layer[l + 1], budget, True)
                else:
                    sel, prot = policy_obj.plan(l + 1, ranks[t][l], budget, False)
                if mode == "pred0":
                    policy_obj.plan_only(l + 1, sel)
                elif isinstance(policy_obj, P.SlotPolicy):
                    dropped = {e for e in sel if drop and (policy_obj.step + e) % drop == 0}
                    policy_obj.prefetch(l + 1, sel, prot, dropped)
                else:
                    policy_obj.prefetch(l + 1, sel, prot, drop)
        if isinstance(policy_obj, P.SlotPolicy):
            policy_obj.step += 1
        else:
            policy_obj.end_step()
            policy_obj.check()                 # structural invariants of the library's table after every step


@pytest.mark.parametrize("mode,S,budget,nb,plain,drop", [
    ("adapter", 4, 2, 1, False, 0), ("adapter", 8, 3, 1, True, 0), ("hint", 6, 2, 1, False, 0),
    ("pred0", 4, 2, 1, False, 0), ("on_demand", 5, 0, 1, False, 0), ("adapter", 5, 2, 7, False, 0),
    ("adapter", 3, 4, 9, False, 3), ("hint", 16, 8, 4, False, 0), ("adapter", 16, 1, 1, False, 2),
])
def test_slot_table_matches_policy_oracle(mode, S, budget, nb, plain, drop):
    L, n, K, steps = 3, 24, 3, 80
    rng = np.random.default_rng(hash((mode, S, budget, nb)) % (1 << 31))
    trace, ranks = [], []
    for _ in range(steps):
        trace.append([sorted({int(e) for _ in range(nb) for e in rng.permutation(n)[:K]}) for _ in range(L)])
        ranks.append([[int(e) for e in rng.permutation(n)] for _ in range(L)])
    ref = P.SlotPolicy(L, n, S, plain)
    sim = B.Sim(L, n, S, plain)
    drive(ref, trace, ranks, L, budget, mode, drop)
    drive(sim, trace, ranks, L, budget, mode, drop)
    assert sim.events() == ref.events
    st = sim.stats()
    for k in ("hits", "hits_prefetched", "misses", "evictions", "wasted", "prefetch_issued", "touches",
              "waves", "planned"):
        assert st[k] == getattr(ref.stats, k), k
    for l in range(L):
        assert sim.slot_table(l) == ref.pools[l].slot_expert
    sim.close()


def test_sim_rejects_bad_arguments():
    sim = B.Sim(2, 8, 3)
    with pytest.raises(B.SpmError):
        sim.demand(5, [1])
    with pytest.raises(B.SpmError):
        sim.demand(0, [99])
    with pytest.raises(B.SpmError):
        sim.plan(1, [0, 1, 8], 2)
    sim.close()


def test_checkpoint_words_match_the_oracle_state_and_resume_identically():
    # export after a run = the oracle's table word for word; a fresh table that imports it and is
    # driven on gives the events an uninterrupted table gives
    L, n, K, S, budget, steps = 3, 24, 3, 6, 2, 60
    rng = np.random.default_rng(11)
    trace = [[sorted({int(e) for e in rng.permutation(n)[:K]}) for _ in range(L)] for _ in range(steps)]
    ranks = [[[int(e) for e in rng.permutation(n)] for _ in range(L)] for _ in range(steps)]
    ref = P.SlotPolicy(L, n, S, False)
    sim = B.Sim(L, n, S, False)
    half = steps // 2
    drive(ref, trace[:half], ranks[:half], L, budget, "adapter")
    drive(sim, trace[:half], ranks[:half], L, budget, "adapter")
    words = sim.export_state()
    assert words.size == 2 + 4 * L * S and words[0] == ref.tick and words[1] == ref.step == half
    for l in range(L):
        for s in range(S):
            w = words[2 + 4 * (l * S + s):6 + 4 * (l * S + s)]
            p = ref.pools[l]
            assert list(w) == [p.slot_expert[s], p.slot_tick[s], p.slot_origin[s], p.slot_used[s]], (l, s)
    resumed = B.Sim(L, n, S, False)
    resumed.import_state(words)
    n_before = len(sim.events())
    drive(sim, trace[half:], ranks[half:], L, budget, "adapter")
    drive(resumed, trace[half:], ranks[half:], L, budget, "adapter")
    assert resumed.events() == sim.events()[n_before:]
    assert [resumed.slot_table(l) for l in range(L)] == [sim.slot_table(l) for l in range(L)]
    # invalid states are refused and leave the table as it was
    keep = resumed.export_state()
    for bad in (words[:-1], np.concatenate((words, [0])), np.where(np.arange(words.size) == 2, n, words),
                np.where(np.arange(words.size) == 3, words[0] + 1, words)):
        with pytest.raises(B.SpmError):
            resumed.import_state(bad)
    dup = words.copy()
    dup[2 + 4] = dup[2]                    # the same expert in two slots of layer 0
    if dup[2] >= 0:
        with pytest.raises(B.SpmError):
            resumed.import_state(dup)
    assert np.array_equal(resumed.export_state(), keep)
    for x in (sim, resumed):
        x.close()
