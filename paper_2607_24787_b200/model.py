"""Device-side setup of an offloaded MoE decode context: allocates HBM, the pinned expert store and
the two CUDA streams with torch (plumbing only), packs expert weights into the library's blob
layout and hands raw pointers to the C ABI. No decode arithmetic happens in Python.
"""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from . import binding as B


def pack_experts(gate: torch.Tensor, up: torch.Tensor, down: torch.Tensor) -> torch.Tensor:
    """Logical matrices -> packed blobs (layout documented in include/spm.h).

    gate, up: [ne, I, D]; down: [ne, D, I]. Returns [ne, I, 3, D] contiguous, same dtype:
    blob row j = (gate[j], up[j], column j of down).
    """
    return torch.stack((gate, up, down.transpose(1, 2)), dim=2).contiguous()


def pack_experts_q4(gate, up, down_t) -> torch.Tensor:
    """4-bit experts -> packed blobs. Each argument is (q uint8 [ne, I, D] in 0..15, scale fp16
    [ne, I, D/32]); `down_t` row j is column j of W_down. Returns uint8 [ne, I, 3, D/2 + D/16]:
    per row D/2 bytes of nibbles (element 2b low, 2b+1 high) then the D/32 fp16 scales."""
    rows = []
    for q, scale in (gate, up, down_t):
        nib = (q[..., 0::2] | (q[..., 1::2] << 4)).to(torch.uint8)
        sc = scale.contiguous().view(torch.uint8).reshape(*scale.shape[:-1], scale.shape[-1] * 2)
        rows.append(torch.cat((nib, sc), dim=-1))
    return torch.stack(rows, dim=2).contiguous()


class PinnedStore:
    """Page-locked host buffer from spm_host_alloc, viewed as a flat uint8 torch tensor."""

    def __init__(self, nbytes: int):
        self.nbytes = nbytes
        self.ptr = B.spm_host_alloc(nbytes)
        self._raw = (C.c_ubyte * nbytes).from_address(self.ptr)
        self.tensor = torch.frombuffer(self._raw, dtype=torch.uint8)

    def close(self):
        if self.ptr:
            self.tensor = None
            self._raw = None
            B.spm_host_free(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class OffloadedMoE:
    """Owns the buffers of one decode context and forwards to the spm_* entry points.

    gamma [L, D] fp32; router_w [L, n, D]; adapter_a [L-1, r, D]; adapter_b [L-1, n, r] (device
    tensors of the weight dtype); shared_blobs [L, n_shared, I, 3, D] device or None;
    store: PinnedStore holding [L, n] packed expert blobs.
    """

    def __init__(self, *, n_layers, hidden, n_experts, inter, top_k, n_shared, adapter_rank, dtype,
                 renormalize, rms_eps, max_batch, slots, budget, gamma, router_w, adapter_a, adapter_b,
                 shared_blobs, store: PinnedStore, device="cuda:0", store_layers=0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: there is no CPU implementation of this path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.L, self.D, self.n, self.I, self.K = n_layers, hidden, n_experts, inter, top_k
        self.n_shared, self.r, self.slots, self.max_batch = n_shared, adapter_rank, slots, max_batch
        self.cfg = B.make_cfg(n_layers, hidden, n_experts, inter, top_k, n_shared, adapter_rank,
                              {"bf16": B.DTYPE_BF16, torch.bfloat16: B.DTYPE_BF16, "q4": B.DTYPE_Q4}.get(dtype, B.DTYPE_FP32),
                              int(renormalize), max_batch, rms_eps)
        self.blob_bytes = B.spm_expert_blob_bytes(self.cfg)
        self.store_layers = store_layers if 0 < store_layers < n_layers else n_layers
        assert store.nbytes >= self.store_layers * n_experts * self.blob_bytes
        self._keep = [gamma, router_w, adapter_a, adapter_b, shared_blobs, store]
        self.store = store
        self.arena = torch.empty(B.spm_query_arena(self.cfg, slots) + 256, dtype=torch.uint8, device=self.device)
        arena_ptr = (self.arena.data_ptr() + 255) // 256 * 256
        self.compute = torch.cuda.Stream(self.device)
        self.copy = torch.cuda.Stream(self.device)
        buf = B.Buffers(gamma.data_ptr(), router_w.data_ptr(),
                        adapter_a.data_ptr() if adapter_a is not None else None,
                        adapter_b.data_ptr() if adapter_b is not None else None,
                        shared_blobs.data_ptr() if shared_blobs is not None else None,
                        store.ptr, arena_ptr, self.arena.numel() - 256,
                        self.compute.cuda_stream, self.copy.cuda_stream,
                        0 if self.store_layers == n_layers else self.store_layers)
        torch.cuda.synchronize(self.device)
        self.ctx = B.spm_init(self.cfg, slots, budget, buf)

    def close(self):
        if getattr(self, "ctx", None):
            B.spm_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- per-call entry points (device tensors in, numpy for host-visible results) ----
    def router_topk(self, layer, h: torch.Tensor, want_logits=False):
        nb = h.shape[0]
        x = torch.empty_like(h)
        w = torch.empty(nb, self.K, dtype=torch.float32, device=self.device)
        logits = torch.empty(nb, self.n, dtype=torch.float32, device=self.device) if want_logits else None
        ids = np.empty((nb, self.K), np.int32)
        B.spm_router_topk(self.ctx, layer, h, nb, x, ids, w, logits)
        return x, ids, w, logits

    def adapter_predict(self, layer, x_norm: torch.Tensor):
        scores = np.empty(self.n, np.float32)
        order = np.empty(self.n, np.int32)
        B.spm_adapter_predict(self.ctx, layer, x_norm, x_norm.shape[0], scores, order)
        return scores, order

    def budget_select(self, target_layer, order, budget=-1, protect_all=False):
        return B.spm_budget_select(self.ctx, target_layer, order, budget, protect_all)

    def prefetch_async(self, target_layer, ids):
        return B.spm_prefetch_async(self.ctx, target_layer, ids)

    def moe_ffn(self, layer, x_norm, ids, w, h_inout):
        B.spm_moe_ffn(self.ctx, layer, x_norm, ids, w, x_norm.shape[0], h_inout)

    def decode_step(self, h_in: torch.Tensor, h_out: torch.Tensor | None = None):
        if h_out is None:
            h_out = torch.empty_like(h_in)
        B.spm_decode_step(self.ctx, h_in, h_in.shape[0], h_out)
        return h_out

    def decode_step_host(self, h_in_host: torch.Tensor, h_out_host: torch.Tensor):
        B.spm_decode_step_host(self.ctx, h_in_host, h_in_host.shape[0], h_out_host)
        return h_out_host

    # ---- control / accounting --------------------------------------------
    def set_policy(self, p): B.spm_set_policy(self.ctx, p)
    def set_budget(self, b): B.spm_set_budget(self.ctx, b)
    def get_budget(self): return B.spm_get_budget(self.ctx)
    def set_plain_lru(self, on): B.spm_set_plain_lru(self.ctx, on)
    def set_timing(self, on): B.spm_set_timing(self.ctx, on)
    def set_ffn_ctas(self, g): B.spm_set_ffn_ctas(self.ctx, g)
    def set_batched_path(self, mode): B.spm_set_batched_path(self.ctx, mode)
    def set_hint_trace(self, hint): B.spm_set_hint_trace(self.ctx, hint)
    def set_drop_modulo(self, m): B.spm_set_drop_modulo(self.ctx, m)
    def set_attention_stub_us(self, us): B.spm_set_attention_stub_us(self.ctx, us)
    def set_device_wait(self, on): B.spm_set_device_wait(self.ctx, on)
    def set_host_free(self, on): B.spm_set_host_free(self.ctx, on)
    def set_graph_replay(self, on): B.spm_set_graph_replay(self.ctx, on)
    def set_copy_delay_us(self, us): B.spm_set_copy_delay_us(self.ctx, us)
    def profile_window(self): return B.spm_profile_window(self.ctx)
    def get_profile(self): return B.spm_get_profile(self.ctx)
    def measure_read_bandwidth(self, nbytes, reps=5): return B.spm_measure_read_bandwidth(self.ctx, nbytes, reps)
    def time_ffn_kernel(self, first_layer, x_norm, ids, w, chained=True): return B.spm_time_ffn_kernel(self.ctx, first_layer, x_norm, ids, w, chained)
    def set_event_log_limit(self, n): B.spm_set_event_log_limit(self.ctx, n)
    def set_device_wait_limit_us(self, us): B.spm_set_device_wait_limit_us(self.ctx, us)
    def test_withhold_arrivals(self, count): B.spm_test_withhold_arrivals(self.ctx, count)
    def cache_reset(self): B.spm_cache_reset(self.ctx)
    def check_invariants(self, with_device=True): B.spm_check_invariants(self.ctx, with_device)
    def cache_export(self): return B.spm_cache_export(self.ctx)
    def cache_import(self, state): B.spm_cache_import(self.ctx, state)
    def reset_stats(self): B.spm_reset_stats(self.ctx)
    def stats(self): return B.spm_get_stats(self.ctx)
    def layer_times(self): return B.spm_get_layer_times(self.ctx, self.L)
    def events(self): return B.spm_get_events(self.ctx)
    def slot_table(self, layer): return B.spm_get_slot_table(self.ctx, layer, self.slots)
    def synchronize(self): B.spm_synchronize(self.ctx)
