"""Builds an OffloadedMoE from the counter-based synthetic generator (module `synth`): weights
are generated on the GPU layer by layer, packed, and copied down into the pinned expert store."""
from __future__ import annotations

import torch

import synth

from .adapter_fit import reduced_rank_fit, svd_adapter
from .model import OffloadedMoE, PinnedStore, pack_experts, pack_experts_q4


def packed_experts(cfg: synth.ModelCfg, layer: int, experts, device) -> torch.Tensor:
    """Packed blobs (flat uint8 per expert) of the listed experts of one layer."""
    if cfg.dtype == "q4":
        g, u, d = synth.expert_q4(cfg, layer, experts, device=device)
        return pack_experts_q4(g, u, d)
    g, u, d = synth.expert_matrices(cfg, layer, experts, device=device)
    return pack_experts(g, u, d).view(torch.uint8)


def fill_store(cfg: synth.ModelCfg, store: PinnedStore, device, chunk: int = 32, layers=None):
    """Generate and pack every routed expert of the first `layers` (default all) layers into the pinned host store."""
    blob = cfg.expert_bytes
    for l in range(cfg.n_layers if layers is None else layers):
        for e0 in range(0, cfg.n_experts, chunk):
            es = range(e0, min(e0 + chunk, cfg.n_experts))
            packed = packed_experts(cfg, l, es, device).reshape(-1)
            off = (l * cfg.n_experts + e0) * blob
            store.tensor[off:off + packed.numel()].copy_(packed)
            del packed
    torch.cuda.synchronize(device)


def collect_router_io(m: OffloadedMoE, H_dev: torch.Tensor):
    """Calibration pass for fitted adapters: decodes the rows of H_dev [steps, 1, D] layer by layer
    through the stand-alone entry points and records, per layer, the router input x and the native
    router logits z. Returns (X [L, steps, D], Z [L, steps, n]) fp32 on the device."""
    steps = H_dev.shape[0]
    X = torch.empty(m.L, steps, m.D, dtype=torch.float32, device=m.device)
    Z = torch.empty(m.L, steps, m.n, dtype=torch.float32, device=m.device)
    for s in range(steps):
        h = H_dev[s].clone()
        torch.cuda.synchronize(m.device)
        for l in range(m.L):
            x, ids, w, logits = m.router_topk(l, h, want_logits=True)
            m.moe_ffn(l, x, ids, w, h)
            m.synchronize()
            X[l, s].copy_(x[0])
            Z[l, s].copy_(logits[0])
    torch.cuda.synchronize(m.device)
    return X, Z


def fitted_adapters(X: torch.Tensor, Z: torch.Tensor, rank: int, dtype: torch.dtype, ridge: float = 1e-3):
    """Reduced-rank regression of layer l+1's router logits on layer l's router input, per layer.
    Returns (A [L-1, rank, D], B_up [L-1, n, rank]) in `dtype`."""
    a_all, b_all = [], []
    for l in range(X.shape[0] - 1):
        a, b = reduced_rank_fit(X[l], Z[l + 1], rank, ridge)
        a_all.append(a.to(dtype))
        b_all.append(b.to(dtype))
    return torch.stack(a_all).contiguous(), torch.stack(b_all).contiguous()


def build_from_synth(cfg: synth.ModelCfg, slots=None, budget=None, max_batch=None, device="cuda:0",
                     store: PinnedStore | None = None, adapter="random", store_layers: int = 0) -> OffloadedMoE:
    """Random-init model of the configuration's shape, experts offloaded to pinned host memory.

    adapter="random": the configuration's N(0, 0.02) rank-r adapters. adapter="gate_reuse": a
    training-free stand-in for trained adapters, A^l = W_r^{l+1} and Bup = identity (rank n), i.e.
    the next layer's own gate applied to this layer's router input. adapter="svd": the rank-r
    truncated SVD of W_r^{l+1}. adapter=(A, B_up): given tensors [L-1, r, D] and [L-1, n, r], e.g.
    from fitted_adapters(). All of these are data only: the same kernels run them.
    """
    dev = torch.device(device)
    L = cfg.n_layers
    gamma = torch.ones(L, cfg.hidden, dtype=torch.float32, device=dev)
    router = torch.stack([synth.router_w(cfg, l, dev) for l in range(L)]).contiguous()
    rank = cfg.adapter_rank
    if isinstance(adapter, tuple) and L > 1:
        a, b = (t.to(device=dev, dtype=router.dtype).contiguous() for t in adapter)
        rank = a.shape[1]
        assert a.shape == (L - 1, rank, cfg.hidden) and b.shape == (L - 1, cfg.n_experts, rank)
    elif adapter == "svd" and L > 1:
        pairs = [svd_adapter(router[l + 1], rank) for l in range(L - 1)]
        a = torch.stack([p[0] for p in pairs]).to(router.dtype).contiguous()
        b = torch.stack([p[1] for p in pairs]).to(router.dtype).contiguous()
    elif adapter == "gate_reuse" and L > 1:
        rank = cfg.n_experts
        a = router[1:].clone().contiguous()
        b = torch.eye(cfg.n_experts, dtype=router.dtype, device=dev).expand(L - 1, -1, -1).contiguous()
    elif L > 1:
        a = torch.stack([synth.adapter_a(cfg, l, dev) for l in range(L - 1)]).contiguous()
        b = torch.stack([synth.adapter_b(cfg, l, dev) for l in range(L - 1)]).contiguous()
    else:
        a = b = None
    shared = None
    if cfg.n_shared:
        per_layer = []
        for l in range(L):
            per_layer.append(packed_experts(cfg, l, range(cfg.n_experts, cfg.n_experts + cfg.n_shared), dev))
        shared = torch.stack(per_layer).contiguous()
    # store_layers < L: a host that cannot pin the whole store keeps only that many layers of experts;
    # layer l then reads the blobs of layer l % store_layers (same sizes and traffic, repeated weights)
    kl = store_layers if 0 < store_layers < L else L
    if store is None:
        store = PinnedStore(kl * cfg.n_experts * cfg.expert_bytes)
        fill_store(cfg, store, dev, layers=kl)
    return OffloadedMoE(n_layers=L, hidden=cfg.hidden, n_experts=cfg.n_experts, inter=cfg.inter,
                        top_k=cfg.top_k, n_shared=cfg.n_shared, adapter_rank=rank,
                        dtype=cfg.dtype, renormalize=cfg.renormalize, rms_eps=cfg.rms_eps,
                        max_batch=cfg.batch if max_batch is None else max_batch,
                        slots=cfg.slots if slots is None else slots,
                        budget=cfg.budget if budget is None else budget,
                        gamma=gamma, router_w=router, adapter_a=a, adapter_b=b, shared_blobs=shared,
                        store=store, device=device, store_layers=kl)
