"""Counter-based synthetic inputs for the offloaded-MoE decode workloads.

Every weight element is a pure function of (seed, tensor tag, layer, expert,
flat index), so any single matrix of the 54 GiB Qwen3-shaped store can be
regenerated on its own, on the CPU or on a GPU, with identical bits:

    u16   = top 16 bits of a 32-bit integer hash of the counter
    value = round_to_dtype(sigma * Phi^-1((u16 + 0.5) / 65536))

i.e. inverse-CDF sampling of N(0, sigma^2) on a 65536-point grid (tails end at
about +-4.3 sigma). The quantile table is always computed on the CPU in fp64 and
then moved, so a CUDA device and the host see the same table. Only integer ops
and a table lookup run on the device.

Token ids follow a bounded Zipf law, P(id = i) proportional to (i+1)^-1.1 for
i in [0, vocab), drawn by inverse CDF (float64 cumulative sums) from
numpy's PCG64 stream.

Nothing in this module computes any part of the decode step.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from functools import lru_cache

import numpy as np
import torch

_M32 = 0xFFFFFFFF

TAG_EMB = 1
TAG_ROUTER = 2
TAG_ADAPTER_A = 3
TAG_ADAPTER_B = 4
TAG_GATE = 5
TAG_UP = 6
TAG_DOWN = 7


@dataclass(frozen=True)
class ModelCfg:
    """Shape and workload description of one synthetic decode configuration."""

    name: str
    n_layers: int
    hidden: int
    n_experts: int
    inter: int
    top_k: int
    n_shared: int
    adapter_rank: int
    dtype: str  # "fp32" / "bf16": storage type of every weight matrix; "q4": experts 4-bit, the rest bf16
    slots: int  # routed-expert cache slots per layer
    budget: int  # prefetch budget M_max; -1 = derive from the profiled window
    batch: int  # sequences decoded per step
    steps: int
    vocab: int
    seed: int
    renormalize: int = 1
    rms_eps: float = 1e-6
    sigma_w: float = 0.02
    zipf_a: float = 1.1

    def replace(self, **kw) -> "ModelCfg":
        return dataclasses.replace(self, **kw)

    @property
    def elem_bytes(self) -> int:
        """Bytes per element of the router / adapter matrices."""
        return 4 if self.dtype == "fp32" else 2

    @property
    def expert_bytes(self) -> int:
        if self.dtype == "q4":      # 32 weights = 16 bytes of nibbles + one fp16 scale: 4.5 bit per weight
            return 3 * self.inter * (self.hidden // 2 + self.hidden // 16)
        return 3 * self.hidden * self.inter * self.elem_bytes

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16


CONFIGS = {
    # tiny fp32 parity configuration
    "tiny": ModelCfg("tiny", 2, 256, 16, 128, 2, 0, 8, "fp32", 4, 2, 1, 64, 1024, 0),
    # Qwen3-VL-30B-A3B-shaped text MoE decode
    "qwen3": ModelCfg("qwen3", 48, 2048, 128, 768, 8, 0, 16, "bf16", 16, -1, 1, 256, 151936, 1),
    # DeepSeek-VL2-Tiny-shaped MoE decode, 2 always-resident shared experts
    "dsvl2": ModelCfg("dsvl2", 12, 1280, 64, 896, 6, 2, 16, "bf16", 8, -1, 1, 256, 129280, 2),
    # the same two shapes with 4-bit experts (the paper's on-device setting: 1.94 MB per DeepSeek expert)
    "qwen3_q4": ModelCfg("qwen3_q4", 48, 2048, 128, 768, 8, 0, 16, "q4", 16, -1, 1, 256, 151936, 1),
    "dsvl2_q4": ModelCfg("dsvl2_q4", 12, 1280, 64, 896, 6, 2, 16, "q4", 8, -1, 1, 256, 129280, 2),
    # budget / cache sweep on the Qwen3 shape (budget and slots overridden per cell)
    "sweep": ModelCfg("sweep", 48, 2048, 128, 768, 8, 0, 16, "bf16", 16, 1, 1, 512, 151936, 3),
    # batched decode on the Qwen3 shape
    "batched": ModelCfg("batched", 48, 2048, 128, 768, 8, 0, 16, "bf16", 32, -1, 64, 128, 151936, 4),
    # ... and with 4-bit experts
    "batched_q4": ModelCfg("batched_q4", 48, 2048, 128, 768, 8, 0, 16, "q4", 32, -1, 64, 128, 151936, 4),
}


def get_config(name: str, **overrides) -> ModelCfg:
    cfg = CONFIGS[name]
    return cfg.replace(**overrides) if overrides else cfg


# --------------------------------------------------------------------------
# integer hash
# --------------------------------------------------------------------------
def _mix32_py(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Same mixer on an int64 tensor whose values lie in [0, 2^32)."""
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32  # may wrap in int64; the low 32 bits are exact
    x = x ^ (x >> 16)
    return x


def _key(seed: int, tag: int, layer: int, expert: int) -> tuple[int, int]:
    k = _mix32_py(seed * 0x9E3779B1 + tag * 0x85EBCA77 + layer * 0xC2B2AE3D
                  + expert * 0x27D4EB2F + 0x165667B1)
    k2 = _mix32_py(k ^ 0x5BD1E995)
    return k, k2


def hash_u16(seed: int, tag: int, layer: int, experts, count: int, device="cpu") -> torch.Tensor:
    """[len(experts), count] int64 values in [0, 65536)."""
    assert 0 < count < (1 << 32)
    keys = [_key(seed, tag, layer, int(e)) for e in experts]
    k1 = torch.tensor([k[0] for k in keys], dtype=torch.int64, device=device).unsqueeze(1)
    k2 = torch.tensor([k[1] for k in keys], dtype=torch.int64, device=device).unsqueeze(1)
    idx = torch.arange(count, dtype=torch.int64, device=device).unsqueeze(0)
    h = _mix32(idx ^ k1)
    h = _mix32((h + k2) & _M32)
    return h >> 16


@lru_cache(maxsize=None)
def normal_table() -> torch.Tensor:
    """fp64 standard-normal quantiles at (i + 0.5) / 65536, always built on the CPU."""
    p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    return torch.special.ndtri(p)


@lru_cache(maxsize=None)
def _table_for(sigma: float, dtype: torch.dtype, device: str) -> torch.Tensor:
    t = (normal_table() * sigma).to(torch.float32)
    if dtype == torch.bfloat16:
        t = t.to(torch.bfloat16)  # round to nearest even
    return t.to(device)


def synth_normal(seed: int, tag: int, layer: int, experts, count: int, sigma: float,
                 dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """[len(experts), count] tensor of `dtype`, N(0, sigma^2) on the quantile grid."""
    u = hash_u16(seed, tag, layer, experts, count, device)
    return _table_for(float(sigma), dtype, str(device))[u]


# --------------------------------------------------------------------------
# model tensors (logical layouts; all row-major)
# --------------------------------------------------------------------------
def router_w(cfg: ModelCfg, layer: int, device="cpu") -> torch.Tensor:
    """Gate matrix W_r of layer `layer`: [n_experts, hidden]."""
    return synth_normal(cfg.seed, TAG_ROUTER, layer, [0], cfg.n_experts * cfg.hidden,
                        cfg.sigma_w, cfg.torch_dtype, device).view(cfg.n_experts, cfg.hidden)


def adapter_a(cfg: ModelCfg, layer: int, device="cpu") -> torch.Tensor:
    """Adapter down-projection of the pair (layer, layer+1): [rank, hidden]."""
    return synth_normal(cfg.seed, TAG_ADAPTER_A, layer, [0], cfg.adapter_rank * cfg.hidden,
                        cfg.sigma_w, cfg.torch_dtype, device).view(cfg.adapter_rank, cfg.hidden)


def adapter_b(cfg: ModelCfg, layer: int, device="cpu") -> torch.Tensor:
    """Adapter up-projection of the pair (layer, layer+1): [n_experts, rank]."""
    return synth_normal(cfg.seed, TAG_ADAPTER_B, layer, [0], cfg.n_experts * cfg.adapter_rank,
                        cfg.sigma_w, cfg.torch_dtype, device).view(cfg.n_experts, cfg.adapter_rank)


Q4_GROUP = 32


def quantize_q4(w: torch.Tensor):
    """Symmetric 4-bit quantisation along the last dimension in groups of 32 (input preparation).

    Returns (q uint8 in 0..15, scale fp16) with value = scale * (q - 8); scale = max|w| / 7 of the
    group, rounded to fp16 (1 where the group is all zero)."""
    g = w.to(torch.float32).reshape(*w.shape[:-1], w.shape[-1] // Q4_GROUP, Q4_GROUP)
    scale = (g.abs().amax(dim=-1) / 7.0).to(torch.float16)
    scale = torch.where(scale == 0, torch.ones_like(scale), scale)
    q = torch.clamp(torch.round(g / scale.to(torch.float32).unsqueeze(-1)) + 8, 0, 15).to(torch.uint8)
    return q.reshape(w.shape), scale


def dequantize_q4(q: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """fp32 values scale * (q - 8); exact (an fp16 scale times a 4-bit integer fits fp32)."""
    g = q.to(torch.float32).reshape(*q.shape[:-1], q.shape[-1] // Q4_GROUP, Q4_GROUP) - 8.0
    return (g * scale.to(torch.float32).unsqueeze(-1)).reshape(q.shape)


def expert_q4(cfg: ModelCfg, layer: int, experts, device="cpu"):
    """4-bit experts: ((q, scale) of gate[ne, I, D], of up[ne, I, D], of down^T[ne, I, D]).

    down^T row j is column j of W_down, so its quantisation groups run along the hidden dimension."""
    experts = list(experts)
    ne, I, D = len(experts), cfg.inter, cfg.hidden
    out = []
    for tag in (TAG_GATE, TAG_UP, TAG_DOWN):
        w = synth_normal(cfg.seed, tag, layer, experts, I * D, cfg.sigma_w, torch.bfloat16, device).view(ne, I, D)
        out.append(quantize_q4(w))
    return tuple(out)


def expert_matrices(cfg: ModelCfg, layer: int, experts, device="cpu"):
    """(gate[ne, I, D], up[ne, I, D], down[ne, D, I]) for the listed experts.

    Routed experts are 0..n_experts-1; shared expert s is index n_experts + s.
    With 4-bit experts these are the de-quantised fp32 values.
    """
    experts = list(experts)
    if cfg.dtype == "q4":
        (gq, gs), (uq, us), (dq, dsc) = expert_q4(cfg, layer, experts, device)
        return dequantize_q4(gq, gs), dequantize_q4(uq, us), dequantize_q4(dq, dsc).transpose(1, 2).contiguous()
    ne, I, D = len(experts), cfg.inter, cfg.hidden
    g = synth_normal(cfg.seed, TAG_GATE, layer, experts, I * D, cfg.sigma_w, cfg.torch_dtype, device)
    u = synth_normal(cfg.seed, TAG_UP, layer, experts, I * D, cfg.sigma_w, cfg.torch_dtype, device)
    d = synth_normal(cfg.seed, TAG_DOWN, layer, experts, D * I, cfg.sigma_w, cfg.torch_dtype, device)
    return g.view(ne, I, D), u.view(ne, I, D), d.view(ne, D, I)


def embedding_rows(cfg: ModelCfg, tokens, device="cpu") -> torch.Tensor:
    """fp32 [len(tokens), hidden]: rows of the N(0,1) embedding table (stored in cfg.dtype)."""
    toks = [int(t) for t in np.asarray(tokens).reshape(-1)]
    uniq = sorted(set(toks))
    rows = synth_normal(cfg.seed, TAG_EMB, 0, uniq, cfg.hidden, 1.0, cfg.torch_dtype, device)
    pos = {t: i for i, t in enumerate(uniq)}
    sel = torch.tensor([pos[t] for t in toks], dtype=torch.int64, device=device)
    return rows[sel].to(torch.float32)


# --------------------------------------------------------------------------
# token stream
# --------------------------------------------------------------------------
def zipf_probs(vocab: int, a: float = 1.1) -> np.ndarray:
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-a)
    return w / w.sum()


def zipf_tokens(cfg: ModelCfg, steps: int | None = None, batch: int | None = None,
                stream: int = 0) -> np.ndarray:
    """int64 [steps, batch] token ids, drawn row-major from one PCG64 stream.

    `stream` selects an independent sequence (one per data-parallel replica).
    """
    steps = cfg.steps if steps is None else steps
    batch = cfg.batch if batch is None else batch
    cdf = np.cumsum(zipf_probs(cfg.vocab, cfg.zipf_a))
    cdf[-1] = 1.0
    seed = cfg.seed if stream == 0 else [cfg.seed, stream]
    rng = np.random.Generator(np.random.PCG64(seed))
    u = rng.random(steps * batch)
    ids = np.searchsorted(cdf, u, side="right")
    return np.minimum(ids, cfg.vocab - 1).astype(np.int64).reshape(steps, batch)
