"""CPU oracle, math part: the plain definition of one offloaded-MoE decode layer.

TEST INFRASTRUCTURE ONLY. Nothing in the product path may import this module;
it shares no code with the CUDA library and never sees a value produced by it.
Everything here is numpy float64, written out directly from the definitions,
with no blocking, fusion or reordering.

Conventions: layers are 0-based; D hidden size, n routed experts, K experts per
token, I expert intermediate size, r adapter rank. Matrices are row-major
numpy arrays: W_r[n, D], A[r, D], Bup[n, r], W_gate[I, D], W_up[I, D],
W_down[D, I].

Citations are to the paper's sections and equations:
  * native router and Top-K ................ Section 3.1, first equation
  * batch-level demand ..................... Section 3.1, second equation
  * adapter logits z^ = B A x .............. Section 3.2, first equation
  * predicted distribution softmax(z^) ..... Section 3.2, third equation
  * priority aggregation s_e = sum pi^ ..... Section 3.2, fourth equation
  * candidate set Top_M(s) ................. Section 3.2, sixth equation
  * adapter parameter count ................ Section 3.2, last equation
  * ExpertRecall@M / ReadyRecall ........... Section 4.1, "Evaluation Metrics"
The paper names the expert computation only as "MoE FFN computation"; the
SwiGLU form, the RMSNorm in front of the router and the softmax/top-k/renormalise
gate are the workload definition this build was given.

Pinned by tests/test_oracle_math.py (closed forms, brute-force loops on tiny
inputs, library special cases, invariants). No function here is unpinned.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def rmsnorm(h: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """Router input x = h * gamma / sqrt(mean(h^2) + eps) (Section 3.1: x is the router input)."""
    h = np.asarray(h, F64)
    ms = np.mean(h * h)
    return h * np.asarray(gamma, F64) / np.sqrt(ms + eps)


def softmax(z: np.ndarray) -> np.ndarray:
    """softmax with max subtraction (Section 3.2, third equation)."""
    z = np.asarray(z, F64)
    e = np.exp(z - np.max(z))
    return e / np.sum(e)


def rank_desc(v: np.ndarray) -> np.ndarray:
    """Indices sorted by (value descending, index ascending): ties go to the lower id."""
    v = np.asarray(v)
    idx = np.arange(v.shape[0])
    # lexsort: last key is primary
    return np.lexsort((idx, -v)).astype(np.int64)


def top_k(v: np.ndarray, k: int) -> np.ndarray:
    """Top_K of Section 3.1 / Top_M of Section 3.2: first k entries of the descending ranking."""
    return rank_desc(v)[:k]


def router_logits(W_r: np.ndarray, x: np.ndarray) -> np.ndarray:
    """z = W_r x: the native router R^l applied to the router input (Section 3.1)."""
    return np.asarray(W_r, F64) @ np.asarray(x, F64)


def decision_logits(z: np.ndarray) -> np.ndarray:
    """Logits in the precision the Top-K decision is taken in.

    The kernels take the decision on fp32 logits, so the oracle rounds its fp64
    logits to fp32 before ranking them: values that differ only below fp32
    resolution tie, and ties go to the lower id (pinned by
    test_route_decides_in_fp32).
    """
    return np.asarray(z, F64).astype(np.float32)


def route(z: np.ndarray, k: int, renormalize: bool):
    """(ids[K] in rank order, weights[K]) from router logits.

    p = softmax(z); T = Top_K(z) (the same order as Top_K(p));
    w_e = p_e / sum_{j in T} p_j when renormalising, else w_e = p_e.
    """
    p = softmax(z)
    ids = top_k(decision_logits(z), k)
    w = p[ids]
    if renormalize:
        w = w / np.sum(w)
    return ids, w


def near_tie(z: np.ndarray, k: int, tol: float = 1e-5) -> bool:
    """True when the k-th and (k+1)-th largest logits differ by less than tol."""
    z = np.asarray(z, F64)
    if k >= z.shape[0]:
        return False
    order = rank_desc(z)
    return bool(z[order[k - 1]] - z[order[k]] < tol)


def silu(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a, F64)
    return a / (1.0 + np.exp(-a))


def swiglu_expert(W_gate, W_up, W_down, x) -> np.ndarray:
    """One SwiGLU expert: W_down ( silu(W_gate x) * (W_up x) )."""
    x = np.asarray(x, F64)
    g = np.asarray(W_gate, F64) @ x
    u = np.asarray(W_up, F64) @ x
    return np.asarray(W_down, F64) @ (silu(g) * u)


def moe_ffn(x, ids, w, experts, shared=()) -> np.ndarray:
    """y = sum_k w_k * FFN_{ids[k]}(x) + sum over shared experts FFN_s(x) (weight 1).

    `experts(e)` returns (W_gate, W_up, W_down) of routed expert e; `shared` is a
    sequence of such triples.
    """
    x = np.asarray(x, F64)
    y = np.zeros(x.shape[0], F64)
    for e, we in zip(ids, w):
        Wg, Wu, Wd = experts(int(e))
        y = y + float(we) * swiglu_expert(Wg, Wu, Wd, x)
    for Wg, Wu, Wd in shared:
        y = y + swiglu_expert(Wg, Wu, Wd, x)
    return y


def batch_demand(ids_per_token) -> list[int]:
    """T_batch = union over tokens of their Top-K sets (Section 3.1, second equation), ascending ids."""
    s = set()
    for ids in ids_per_token:
        s.update(int(e) for e in ids)
    return sorted(s)


def adapter_logits(A, Bup, x) -> np.ndarray:
    """z^ = Bup (A x) (Section 3.2, first equation; the paper writes B^l for Bup)."""
    u = np.asarray(A, F64) @ np.asarray(x, F64)
    return np.asarray(Bup, F64) @ u


def adapter_scores(A, Bup, X) -> np.ndarray:
    """s_e = sum over the batch's tokens of softmax(z^)_e, summed in token order (Section 3.2)."""
    X = np.asarray(X, F64)
    s = np.zeros(np.asarray(Bup).shape[0], F64)
    for t in range(X.shape[0]):
        s = s + softmax(adapter_logits(A, Bup, X[t]))
    return s


def adapter_param_count(L: int, r: int, D: int, n: int) -> int:
    """(L - 1) r (D + n) (Section 3.2, last equation)."""
    return (L - 1) * r * (D + n)


def expert_recall_at_m(true_ids_per_token, scores, M: int, K: int) -> float:
    """ExpertRecall@M = mean over tokens of |T ∩ Top_M(s)| / K (Section 4.1)."""
    cand = set(int(e) for e in top_k(np.asarray(scores, F64), M))
    tot = 0.0
    for ids in true_ids_per_token:
        tot += len(cand.intersection(int(e) for e in ids)) / K
    return tot / len(true_ids_per_token)


def ready_recall(true_ids_per_token, available, K: int) -> float:
    """ReadyRecall = mean over tokens of |T ∩ A(t_exec)| / K (Section 4.1)."""
    avail = set(int(e) for e in available)
    tot = 0.0
    for ids in true_ids_per_token:
        tot += len(avail.intersection(int(e) for e in ids)) / K
    return tot / len(true_ids_per_token)


def window_budget(window_us: float, t_xfer_us: float) -> int:
    """Raw profiled budget: how many whole expert transfers fit in the overlap window (Section 3.3)."""
    if t_xfer_us <= 0:
        raise ValueError("t_xfer must be positive")
    return int(np.floor(window_us / t_xfer_us))


def run_budget(window_us: float, t_xfer_us: float) -> int:
    """Budget actually used: max(1, raw) so that the prefetch path is exercised."""
    return max(1, window_budget(window_us, t_xfer_us))


def rel_linf(a, b) -> float:
    """max|a-b| / max|b|: the tolerance metric for activations."""
    a = np.asarray(a, F64)
    b = np.asarray(b, F64)
    den = np.max(np.abs(b))
    return float(np.max(np.abs(a - b)) / (den if den > 0 else 1.0))
