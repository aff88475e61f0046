"""Pins for oracle/ref_math.py: closed forms, brute-force loops, library special cases,
invariants and the constants the paper prints. CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ref_math as M

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = v.strip()
    return vals


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_closed_forms():
    D = 7
    g = rng.uniform(0.5, 2.0, D)
    # constant vector c: mean(h^2) = c^2, so x = sign(c) * gamma when eps = 0
    assert np.allclose(M.rmsnorm(np.full(D, -3.0), g, 0.0), -g, rtol=1e-15)
    # all ones with eps: x = gamma / sqrt(1 + eps)
    assert np.allclose(M.rmsnorm(np.ones(D), g, 0.25), g / math.sqrt(1.25), rtol=1e-15)
    # one-hot of magnitude a in D dims: mean square a^2/D
    h = np.zeros(D); h[2] = 4.0
    x = M.rmsnorm(h, np.ones(D), 0.0)
    assert x[2] == pytest.approx(math.sqrt(D)) and np.count_nonzero(x) == 1


def test_rmsnorm_invariants_and_loop():
    D = 33
    h = rng.normal(size=D); g = rng.uniform(0.5, 2.0, D)
    x = M.rmsnorm(h, g, 0.0)
    assert np.mean((x / g) ** 2) == pytest.approx(1.0, rel=1e-14)
    assert np.allclose(M.rmsnorm(5.0 * h, g, 0.0), x, rtol=1e-14)          # scale invariance
    acc = 0.0
    for v in h:
        acc += v * v
    want = [h[i] * g[i] / math.sqrt(acc / D + 1e-6) for i in range(D)]
    assert np.allclose(M.rmsnorm(h, g, 1e-6), want, rtol=1e-14)
    # dropping gamma or eps must be visible
    assert not np.allclose(M.rmsnorm(h, g, 1e-6), M.rmsnorm(h, np.ones(D), 1e-6))
    assert not np.allclose(M.rmsnorm(h, g, 0.5), x)


# ---------------------------------------------------------------- softmax
def test_softmax_closed_forms():
    p = M.softmax(np.array([0.3, -1.2]))
    assert p[0] == pytest.approx(1.0 / (1.0 + math.exp(-1.5)), rel=1e-15)      # two-way = logistic
    assert np.allclose(M.softmax(np.full(5, 17.0)), 0.2)
    z = rng.normal(size=40) * 3
    p = M.softmax(z)
    assert abs(p.sum() - 1.0) < 1e-14
    assert np.allclose(M.softmax(z + 1000.0), p, rtol=1e-12)                    # shift invariance, no overflow
    assert np.allclose(p, torch.softmax(torch.tensor(z), 0).numpy(), rtol=1e-13)
    assert np.allclose(np.log(p[3] / p[9]), z[3] - z[9], rtol=1e-12)


# ---------------------------------------------------------------- ranking / Top-K
def brute_rank(v):
    # full stable sort, written independently: repeated selection of the best remaining
    left = list(range(len(v)))
    out = []
    while left:
        best = left[0]
        for i in left[1:]:
            if v[i] > v[best]:
                best = i
        out.append(best)
        left.remove(best)
    return out


def test_rank_and_topk_bruteforce():
    for trial in range(50):
        n = int(rng.integers(1, 40))
        v = rng.normal(size=n)
        if trial % 3 == 0:
            v = np.round(v)            # many ties
        assert list(M.rank_desc(v)) == brute_rank(v)
        k = int(rng.integers(1, n + 1))
        assert list(M.top_k(v, k)) == brute_rank(v)[:k]


def test_topk_adversarial_ties():
    assert list(M.rank_desc(np.zeros(6))) == [0, 1, 2, 3, 4, 5]
    v = np.array([1.0, 3.0, 2.0, 3.0, 2.0, 0.0])
    assert list(M.rank_desc(v)) == [1, 3, 2, 4, 0, 5]
    assert list(M.top_k(v, 3)) == [1, 3, 2]       # tie at the boundary: lower id wins
    assert M.near_tie(v, 3) and not M.near_tie(v, 2) and not M.near_tie(v, 6)


def test_topk_permutation_metamorphic():
    n, k = 24, 5
    v = rng.normal(size=n)
    perm = rng.permutation(n)
    vp = np.empty(n); vp[perm] = v                # expert e moves to perm[e]
    assert set(M.top_k(vp, k)) == {int(perm[e]) for e in M.top_k(v, k)}


# ---------------------------------------------------------------- route
def test_route_weights():
    z = rng.normal(size=16)
    ids, w = M.route(z, 4, True)
    assert abs(w.sum() - 1.0) < 1e-14 and np.all(np.diff(w) <= 0)
    ids2, w2 = M.route(z, 4, False)
    assert list(ids) == list(ids2)
    p = M.softmax(z)
    assert np.allclose(w2, p[ids]) and np.allclose(w, p[ids] / p[ids].sum())
    # K = n without renormalisation is the dense mixture
    ids3, w3 = M.route(z, 16, False)
    assert sorted(ids3) == list(range(16)) and abs(w3.sum() - 1.0) < 1e-14
    # renormalised top-2: closed form logistic of the logit gap
    ids4, w4 = M.route(z, 2, True)
    gap = z[ids4[0]] - z[ids4[1]]
    assert w4[0] == pytest.approx(1.0 / (1.0 + math.exp(-gap)), rel=1e-13)


# ---------------------------------------------------------------- SwiGLU expert
def test_route_decides_in_fp32():
    """The Top-K decision is taken on logits rounded to fp32 (the precision the kernels decide in):
    logits that differ only below fp32 resolution tie, and ties go to the lower id; logits that
    differ above it do not tie."""
    # 1e-12 apart at the K boundary, the HIGHER id slightly larger in fp64: fp32 rounding makes them
    # equal, so the lower id must win. Ranking the fp64 values would return the higher id instead.
    z = np.array([1.0, 1.0 + 1e-12, -3.0])
    assert np.float32(z[0]) == np.float32(z[1]) and z[1] > z[0]
    ids, w = M.route(z, 1, renormalize=True)
    assert list(ids) == [0] and w[0] == pytest.approx(1.0)
    z = np.array([2.0, 1.0, 1.0 + 1e-12, 0.0])
    ids, _ = M.route(z, 2, renormalize=False)
    assert list(ids) == [0, 1]
    # the weights still come from the fp64 softmax, not from rounded values
    _, w = M.route(np.array([1.0, 1.0 + 1e-12, -3.0]), 2, renormalize=False)
    assert w[1] > w[0]
    # 1e-3 apart: far above fp32 resolution at this magnitude, so no tie and the larger logit wins
    z = np.array([1.0, 1.001, -3.0])
    ids, _ = M.route(z, 1, renormalize=True)
    assert list(ids) == [1]
    z = np.array([2.0, 1.0, 1.001, 0.0])
    ids, _ = M.route(z, 2, renormalize=False)
    assert list(ids) == [0, 2]
    # decision_logits itself: fp32 values, nearest rounding, same shape
    d = M.decision_logits(np.array([1.0 + 1e-12, 1.0 + 2.0 ** -24 + 2.0 ** -40, 0.1]))
    assert d.dtype == np.float32
    assert d[0] == np.float32(1.0) and d[1] == np.float32(1.0 + 2.0 ** -23) and d[2] == np.float32(0.1)


def test_batch_demand_union():
    """T_batch is the union of the tokens' Top-K sets: duplicates counted once, ascending ids."""
    assert M.batch_demand([[5, 1], [1, 9], [9, 5]]) == [1, 5, 9]
    assert M.batch_demand([np.array([7, 3, 3])]) == [3, 7]
    assert M.batch_demand([]) == []
    ids = [rng.permutation(32)[:4] for _ in range(6)]
    want = sorted(set(int(e) for row in ids for e in row))
    assert M.batch_demand(ids) == want and all(isinstance(e, int) for e in want)


def test_swiglu_hand_example():
    # D = 2, I = 1: g = 1, u = 2, silu(1) = 1/(1+e^-1); y = W_down * (silu(g) * u)
    y = M.swiglu_expert([[1.0, 0.0]], [[0.0, 1.0]], [[1.0], [-1.0]], [1.0, 2.0])
    a = 2.0 / (1.0 + math.exp(-1.0))
    assert np.allclose(y, [a, -a], rtol=1e-15)
    assert a == pytest.approx(1.4621171572600098, rel=1e-15)


def test_swiglu_vs_loops_and_library():
    D, I = 12, 5
    Wg, Wu = rng.normal(size=(I, D)), rng.normal(size=(I, D))
    Wd = rng.normal(size=(D, I)); x = rng.normal(size=D)
    want = [0.0] * D
    for j in range(I):
        g = sum(Wg[j][i] * x[i] for i in range(D))
        u = sum(Wu[j][i] * x[i] for i in range(D))
        a = g / (1.0 + math.exp(-g)) * u
        for d in range(D):
            want[d] += Wd[d][j] * a
    got = M.swiglu_expert(Wg, Wu, Wd, x)
    assert np.allclose(got, want, rtol=1e-12)
    F = torch.nn.functional
    xt = torch.tensor(x)
    lib = F.linear(F.silu(F.linear(xt, torch.tensor(Wg))) * F.linear(xt, torch.tensor(Wu)), torch.tensor(Wd))
    assert np.allclose(got, lib.numpy(), rtol=1e-12)
    # swapping gate and up must be visible (silu is applied to the gate only)
    assert not np.allclose(M.swiglu_expert(Wu, Wg, Wd, x), got)
    # zero gate -> silu(0) = 0 -> zero output
    assert np.all(M.swiglu_expert(np.zeros((I, D)), Wu, Wd, x) == 0.0)


def test_moe_ffn_special_cases():
    D, I, n = 10, 4, 6
    Ws = [(rng.normal(size=(I, D)), rng.normal(size=(I, D)), rng.normal(size=(D, I))) for _ in range(n)]
    x = rng.normal(size=D)
    # n = K = 1: the layer is one dense SwiGLU MLP
    y1 = M.moe_ffn(x, [0], [1.0], lambda e: Ws[e])
    assert np.allclose(y1, M.swiglu_expert(*Ws[0], x))
    # identical experts + weights summing to one: routing does not matter
    ids, w = M.route(rng.normal(size=n), 3, True)
    assert np.allclose(M.moe_ffn(x, ids, w, lambda e: Ws[2]), M.swiglu_expert(*Ws[2], x), rtol=1e-13)
    # linear in the routing weights; shared experts enter with weight one
    ya = M.moe_ffn(x, [1, 4], [0.25, 0.75], lambda e: Ws[e], shared=[Ws[5]])
    want = 0.25 * M.swiglu_expert(*Ws[1], x) + 0.75 * M.swiglu_expert(*Ws[4], x) + M.swiglu_expert(*Ws[5], x)
    assert np.allclose(ya, want, rtol=1e-13)


# ---------------------------------------------------------------- adapter
def test_adapter_special_cases():
    D, n = 20, 9
    x = rng.normal(size=D)
    W_next = rng.normal(size=(n, D))
    # r = n, A = next router, Bup = identity: the predictor is "next router applied to x^l"
    assert np.allclose(M.adapter_logits(W_next, np.eye(n), x), M.router_logits(W_next, x), rtol=1e-14)
    # r = 1: z^ = Bup[:,0] * (a . x)
    a = rng.normal(size=(1, D)); b = rng.normal(size=(n, 1))
    assert np.allclose(M.adapter_logits(a, b, x), b[:, 0] * float(a[0] @ x), rtol=1e-14)
    # general r against loops (also catches a transposed operand: shapes r != n != D)
    r = 3
    A = rng.normal(size=(r, D)); B = rng.normal(size=(n, r))
    want = [sum(B[e][q] * sum(A[q][i] * x[i] for i in range(D)) for q in range(r)) for e in range(n)]
    assert np.allclose(M.adapter_logits(A, B, x), want, rtol=1e-12)


def test_adapter_scores_aggregate():
    D, n, r, nb = 16, 7, 2, 5
    A = rng.normal(size=(r, D)); B = rng.normal(size=(n, r)); X = rng.normal(size=(nb, D))
    s = M.adapter_scores(A, B, X)
    assert s.sum() == pytest.approx(nb, rel=1e-13)          # total routing mass = number of tokens
    one = M.adapter_scores(A, B, X[:1])
    assert np.allclose(one, M.softmax(M.adapter_logits(A, B, X[0])))
    assert np.allclose(s, sum(M.adapter_scores(A, B, X[t:t + 1]) for t in range(nb)), rtol=1e-13)
    # zero adapter -> uniform priorities -> ranking is the identity (ties to the lower id)
    s0 = M.adapter_scores(np.zeros((r, D)), B, X)
    assert np.allclose(s0, nb / n) and list(M.rank_desc(s0)) == list(range(n))


def test_adapter_param_count_paper_formula():
    g = read_golden("paper_constants.txt")
    # (L-1) r (D+n), Section 3.2
    assert M.adapter_param_count(2, 8, 256, 16) == 2176
    assert M.adapter_param_count(48, 16, 2048, 128) == 1636352
    assert M.adapter_param_count(12, 16, 1280, 64) == 236544
    # Table 3 prints 0.82 M for the 11-MoE-layer, 64-expert, hidden-1280 model: rank 64 in Mi units
    p = M.adapter_param_count(int(g["dsvl2_moe_layers"]), 64, 1280, int(g["dsvl2_experts"]))
    assert round(p / 2 ** 20, 2) == float(g["dsvl2_adapter_params_M"])


# ---------------------------------------------------------------- metrics, budget
def test_recall_bounds_paper():
    g = read_golden("paper_constants.txt")
    n, K = 32, 8
    ids = [rng.permutation(n)[:K] for _ in range(6)]
    s = rng.random(n)
    for Mc in (4, 8, 10, n):
        r = M.expert_recall_at_m(ids, s, Mc, K)
        assert 0.0 <= r <= min(1.0, Mc / K) + 1e-12           # R@M <= M/K
    assert M.expert_recall_at_m(ids, s, n, K) == 1.0
    # the paper: with K = 8 (6) the maximum R@4 (R@3) is 50 %
    assert 4 / 8 == float(g["max_recall_half_budget"]) and 3 / 6 == float(g["max_recall_half_budget"])
    # perfect scores: mass on the true set -> R@K = 1, and R@(K/2) hits the bound
    mass = np.zeros(n); mass[ids[0]] = np.linspace(1, 2, K)
    assert M.expert_recall_at_m(ids[:1], mass, K, K) == 1.0
    assert M.expert_recall_at_m(ids[:1], mass, K // 2, K) == 0.5
    # ReadyRecall counts available experts
    assert M.ready_recall(ids[:1], ids[0][:2], K) == 2 / K
    assert M.ready_recall(ids[:1], range(n), K) == 1.0


def test_window_budget():
    g = read_golden("paper_constants.txt")
    # Figure 1(b): the window holds about two transfers
    assert M.window_budget(2.3 * 170.0, 170.0) == int(g["window_transfers"])
    assert M.window_budget(13.5, 172.0) == 0 and M.run_budget(13.5, 172.0) == 1
    assert M.window_budget(8 * 10.0 + 1e-9, 10.0) == 8 and M.run_budget(85.0, 10.0) == 8
    with pytest.raises(ValueError):
        M.window_budget(1.0, 0.0)


def test_expert_shape_matches_paper_size():
    g = read_golden("paper_constants.txt")
    # Section 4.1: each 4-bit expert takes 1.94 MB; 3 * 1280 * 896 weights at 4.5 bit (4 bit + fp16 scale per 32)
    nbytes = 3 * 1280 * 896 * 4.5 / 8
    assert round(nbytes / 1e6, 2) == float(g["dsvl2_expert_MB_4bit"])


def test_rel_linf():
    assert M.rel_linf([1.0, 2.0], [1.0, 2.0]) == 0.0
    assert M.rel_linf([1.0, 2.5], [1.0, 2.0]) == 0.25
