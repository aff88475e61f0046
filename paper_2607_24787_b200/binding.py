"""ctypes binding of libspm.so: the same entry points as include/spm.h, argument marshalling only.

Every step of the decode path runs inside the library's CUDA kernels and host runtime; this
module converts torch tensors / numpy arrays to raw pointers and raises on a non-zero status.
There is no fallback: if the shared library is missing or does not load, importing callers fail.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libspm.so")

SPM_OK = 0
ERR_NAMES = {-1: "SPM_ERR_INVALID_ARG", -2: "SPM_ERR_CONFIG", -3: "SPM_ERR_CUDA", -4: "SPM_ERR_TIMEOUT",
             -5: "SPM_ERR_NOT_RESIDENT", -6: "SPM_ERR_STATE", -7: "SPM_ERR_NUMERIC"}
DTYPE_FP32, DTYPE_BF16, DTYPE_Q4 = 0, 1, 2
POLICY_ADAPTER, POLICY_ON_DEMAND, POLICY_HINT_TRACE, POLICY_PRED0, POLICY_NAIVE = 0, 1, 2, 3, 4
POLICIES = {"adapter": 0, "on_demand": 1, "hint_trace": 2, "pred0": 3, "naive": 4}
EVENT_NAMES = {1: "HIT", 2: "HIT_PREFETCHED", 3: "MISS", 4: "EVICT", 5: "EVICT_WASTED", 6: "PREFETCH",
               7: "TOUCH_PRED", 8: "WAVE", 9: "PLAN", 10: "DROPPED"}
MAX_BATCH, MAX_TOPK, MAX_EXPERTS = 64, 16, 1024


class SpmError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


class ModelCfg(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("n_layers", "hidden", "n_experts", "inter", "top_k", "n_shared",
                                         "adapter_rank", "dtype", "renormalize", "max_batch")] + [("rms_eps", C.c_float)]


class Buffers(C.Structure):
    _fields_ = [("rms_gamma", C.c_void_p), ("router_w", C.c_void_p), ("adapter_a", C.c_void_p),
                ("adapter_b", C.c_void_p), ("shared_experts", C.c_void_p), ("host_experts", C.c_void_p),
                ("arena", C.c_void_p), ("arena_bytes", C.c_size_t), ("compute_stream", C.c_void_p),
                ("copy_stream", C.c_void_p), ("host_store_layers", C.c_int32)]


class Event(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("step", "layer", "kind", "expert", "slot")]


class Stats(C.Structure):
    _fields_ = ([(k, C.c_uint64) for k in ("steps", "tokens", "hits", "hits_prefetched", "misses", "evictions",
                                           "wasted", "prefetch_issued", "touches", "waves", "planned", "dropped",
                                           "late_arrivals", "h2d_bytes", "ffn_launches", "kernel_launches")]
                + [("ffn_us", C.c_double), ("ffn_window_us", C.c_double), ("stall_us", C.c_double), ("ready_sum", C.c_double),
                   ("ready_count", C.c_uint64), ("recall_sum", C.c_double), ("recall_count", C.c_uint64),
                   ("host_free_steps", C.c_uint64), ("router_window_us", C.c_double), ("reduce_window_us", C.c_double),
                   ("gap_us", C.c_double), ("recall_at", C.c_double * 3), ("events_dropped", C.c_uint64)])

    def as_dict(self):
        d = {k: getattr(self, k) for k, _ in self._fields_}
        d["recall_at"] = list(d["recall_at"])
        return d


# symbol -> argument types (all return int except spm_last_error)
_P = C.c_void_p
_SIG = {
    "spm_expert_blob_bytes": [C.POINTER(ModelCfg), C.POINTER(C.c_size_t)],
    "spm_query_arena": [C.POINTER(ModelCfg), C.c_int, C.POINTER(C.c_size_t)],
    "spm_init": [C.POINTER(ModelCfg), C.c_int, C.c_int, C.POINTER(Buffers), C.POINTER(_P)],
    "spm_destroy": [_P],
    "spm_router_topk": [_P, C.c_int, _P, C.c_int, _P, _P, _P, _P],
    "spm_adapter_predict": [_P, C.c_int, _P, C.c_int, _P, _P],
    "spm_budget_select": [_P, C.c_int, _P, C.c_int, C.c_int, C.c_int, _P, C.POINTER(C.c_int)],
    "spm_prefetch_async": [_P, C.c_int, _P, C.c_int, C.POINTER(C.c_int)],
    "spm_moe_ffn": [_P, C.c_int, _P, _P, _P, C.c_int, _P],
    "spm_decode_step": [_P, _P, C.c_int, _P],
    "spm_decode_step_host": [_P, _P, C.c_int, _P],
    "spm_set_policy": [_P, C.c_int],
    "spm_set_budget": [_P, C.c_int],
    "spm_get_budget": [_P, C.POINTER(C.c_int)],
    "spm_set_plain_lru": [_P, C.c_int],
    "spm_set_timing": [_P, C.c_int],
    "spm_set_ffn_ctas": [_P, C.c_int],
    "spm_set_batched_path": [_P, C.c_int],
    "spm_set_hint_trace": [_P, _P, _P, C.c_int, C.c_int],
    "spm_set_drop_modulo": [_P, C.c_int],
    "spm_set_deadline_ms": [_P, C.c_int],
    "spm_set_attention_stub_us": [_P, C.c_int],
    "spm_set_device_wait": [_P, C.c_int],
    "spm_set_host_free": [_P, C.c_int],
    "spm_set_graph_replay": [_P, C.c_int],
    "spm_set_copy_delay_us": [_P, C.c_int],
    "spm_profile_window": [_P, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int)],
    "spm_get_profile": [_P, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int)],
    "spm_measure_read_bandwidth": [_P, C.c_size_t, C.c_int, C.POINTER(C.c_double)],
    "spm_time_ffn_kernel": [_P, C.c_int, _P, _P, _P, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)],
    "spm_set_device_wait_limit_us": [_P, C.c_int],
    "spm_set_event_log_limit": [_P, C.c_size_t],
    "spm_test_withhold_arrivals": [_P, C.c_int],
    "spm_cache_reset": [_P],
    "spm_reset_stats": [_P],
    "spm_get_stats": [_P, C.POINTER(Stats)],
    "spm_get_layer_times": [_P, _P, _P, C.POINTER(C.c_uint64)],
    "spm_get_events": [_P, _P, C.c_size_t, C.POINTER(C.c_size_t)],
    "spm_get_slot_table": [_P, C.c_int, _P],
    "spm_synchronize": [_P],
    "spm_ffn_noalloc": [C.POINTER(ModelCfg), _P, C.c_int, _P, _P, C.c_int, _P, _P, _P, C.c_int],
    "spm_host_alloc": [C.c_size_t, C.POINTER(_P)],
    "spm_host_free": [_P],
    "spm_sim_create": [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(_P)],
    "spm_sim_destroy": [_P],
    "spm_plan_grouped_chunks": [C.c_int, C.c_int, C.c_int, _P, C.c_size_t, C.POINTER(C.c_size_t)],
    "spm_sim_demand": [_P, C.c_int, _P, C.c_int, _P, _P, _P, _P, C.POINTER(C.c_int), C.POINTER(C.c_int)],
    "spm_sim_plan": [_P, C.c_int, _P, C.c_int, C.c_int, C.c_int, _P, C.POINTER(C.c_int), _P, C.POINTER(C.c_int)],
    "spm_sim_prefetch": [_P, C.c_int, _P, C.c_int, _P, C.c_int, C.c_int, _P, C.POINTER(C.c_int)],
    "spm_sim_plan_only": [_P, C.c_int, _P, C.c_int],
    "spm_sim_end_step": [_P],
    "spm_sim_events": [_P, _P, C.c_size_t, C.POINTER(C.c_size_t)],
    "spm_sim_stats": [_P, C.POINTER(Stats)],
    "spm_sim_slot_table": [_P, C.c_int, _P],
    "spm_sim_check": [_P],
    "spm_check_invariants": [_P, C.c_int],
    "spm_sim_export": [_P, _P, C.c_size_t, C.POINTER(C.c_size_t)],
    "spm_sim_import": [_P, _P, C.c_size_t],
    "spm_cache_export": [_P, _P, C.c_size_t, C.POINTER(C.c_size_t)],
    "spm_cache_import": [_P, _P, C.c_size_t],
}
EXPORTS = sorted(list(_SIG) + ["spm_last_error"])

_lib = None


def load() -> C.CDLL:
    """Load libspm.so (built in-tree by paper_2607_24787_b200.build). Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2607_24787_b200.build` "
                               "(there is no fallback implementation)")
        lib = C.CDLL(LIB_PATH)
        for name, args in _SIG.items():
            fn = getattr(lib, name)
            fn.argtypes = args
            fn.restype = C.c_int
        lib.spm_last_error.argtypes = [_P]
        lib.spm_last_error.restype = C.c_char_p
        _lib = lib
    return _lib


def _ptr(x):
    """Raw address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


def _check(rc, ctx=None):
    if rc != SPM_OK:
        raise SpmError(rc, load().spm_last_error(ctx).decode())


def make_cfg(n_layers, hidden, n_experts, inter, top_k, n_shared, adapter_rank, dtype, renormalize=1,
             max_batch=1, rms_eps=1e-6) -> ModelCfg:
    return ModelCfg(n_layers, hidden, n_experts, inter, top_k, n_shared, adapter_rank, dtype, renormalize,
                    max_batch, rms_eps)


# ---- entry points, same names as the C ABI ----------------------------------
def spm_expert_blob_bytes(cfg: ModelCfg) -> int:
    out = C.c_size_t()
    _check(load().spm_expert_blob_bytes(C.byref(cfg), C.byref(out)))
    return out.value


def spm_query_arena(cfg: ModelCfg, slots: int) -> int:
    out = C.c_size_t()
    _check(load().spm_query_arena(C.byref(cfg), slots, C.byref(out)))
    return out.value


def spm_init(cfg: ModelCfg, slots: int, budget: int, buffers: Buffers) -> int:
    out = _P()
    _check(load().spm_init(C.byref(cfg), slots, budget, C.byref(buffers), C.byref(out)))
    return out.value


def spm_destroy(ctx):
    _check(load().spm_destroy(ctx))


def spm_router_topk(ctx, layer, h, nb, x_norm, ids: np.ndarray, w, logits=None):
    _check(load().spm_router_topk(ctx, layer, _ptr(h), nb, _ptr(x_norm), _ptr(ids), _ptr(w), _ptr(logits)), ctx)


def spm_adapter_predict(ctx, layer, x_norm, nb, scores: np.ndarray, order: np.ndarray):
    _check(load().spm_adapter_predict(ctx, layer, _ptr(x_norm), nb, _ptr(scores), _ptr(order)), ctx)


def spm_budget_select(ctx, target_layer, order: np.ndarray, budget=-1, protect_all=False) -> np.ndarray:
    order = np.ascontiguousarray(order, np.int32)
    out = np.empty(max(len(order), 1), np.int32)
    cnt = C.c_int()
    _check(load().spm_budget_select(ctx, target_layer, _ptr(order), len(order), budget, int(protect_all),
                                    _ptr(out), C.byref(cnt)), ctx)
    return out[:cnt.value].copy()


def spm_prefetch_async(ctx, target_layer, ids) -> int:
    ids = np.ascontiguousarray(ids, np.int32)
    issued = C.c_int()
    _check(load().spm_prefetch_async(ctx, target_layer, _ptr(ids), len(ids), C.byref(issued)), ctx)
    return issued.value


def spm_moe_ffn(ctx, layer, x_norm, ids: np.ndarray, w, nb, h_inout):
    ids = np.ascontiguousarray(ids, np.int32)
    _check(load().spm_moe_ffn(ctx, layer, _ptr(x_norm), _ptr(ids), _ptr(w), nb, _ptr(h_inout)), ctx)


def spm_decode_step(ctx, h_in, nb, h_out):
    _check(load().spm_decode_step(ctx, _ptr(h_in), nb, _ptr(h_out)), ctx)


def spm_decode_step_host(ctx, h_in_host, nb, h_out_host):
    _check(load().spm_decode_step_host(ctx, _ptr(h_in_host), nb, _ptr(h_out_host)), ctx)


def spm_set_policy(ctx, policy):
    _check(load().spm_set_policy(ctx, POLICIES[policy] if isinstance(policy, str) else policy), ctx)


def spm_set_budget(ctx, budget):
    _check(load().spm_set_budget(ctx, budget), ctx)


def spm_get_budget(ctx) -> int:
    out = C.c_int()
    _check(load().spm_get_budget(ctx, C.byref(out)), ctx)
    return out.value


def spm_set_plain_lru(ctx, on):
    _check(load().spm_set_plain_lru(ctx, int(on)), ctx)


def spm_set_timing(ctx, on):
    _check(load().spm_set_timing(ctx, int(on)), ctx)


def spm_set_ffn_ctas(ctx, ctas):
    _check(load().spm_set_ffn_ctas(ctx, ctas), ctx)


def spm_set_batched_path(ctx, mode):
    _check(load().spm_set_batched_path(ctx, mode), ctx)


def spm_set_hint_trace(ctx, hint):
    """hint[step][layer] = list of expert ids in priority order."""
    n_steps = len(hint)
    L = len(hint[0]) if n_steps else 0
    stride = max(1, max((len(c) for s in hint for c in s), default=1))
    arr = np.full((n_steps, L, stride), -1, np.int32)
    cnt = np.zeros((n_steps, L), np.int32)
    for s, per_layer in enumerate(hint):
        for l, ids in enumerate(per_layer):
            arr[s, l, :len(ids)] = ids
            cnt[s, l] = len(ids)
    arr[arr < 0] = 0
    if arr.size == 0:                      # empty trace: still pass valid pointers
        arr, cnt = np.zeros(1, np.int32), np.zeros(1, np.int32)
    _check(load().spm_set_hint_trace(ctx, _ptr(arr), _ptr(cnt), n_steps, stride), ctx)


def spm_set_drop_modulo(ctx, modulo):
    _check(load().spm_set_drop_modulo(ctx, modulo), ctx)


def spm_set_copy_delay_us(ctx, us):
    _check(load().spm_set_copy_delay_us(ctx, us), ctx)


def spm_set_device_wait(ctx, on):
    _check(load().spm_set_device_wait(ctx, int(on)), ctx)


def spm_set_host_free(ctx, on):
    _check(load().spm_set_host_free(ctx, int(on)), ctx)


def spm_set_graph_replay(ctx, on):
    _check(load().spm_set_graph_replay(ctx, int(on)), ctx)


def spm_set_attention_stub_us(ctx, us):
    _check(load().spm_set_attention_stub_us(ctx, us), ctx)


def spm_set_deadline_ms(ctx, ms):
    _check(load().spm_set_deadline_ms(ctx, ms), ctx)


def spm_profile_window(ctx):
    """(window_us, t_xfer_us, raw budget = floor(window / t_xfer))."""
    w, t, b = C.c_double(), C.c_double(), C.c_int()
    _check(load().spm_profile_window(ctx, C.byref(w), C.byref(t), C.byref(b)), ctx)
    return w.value, t.value, b.value


def spm_get_profile(ctx):
    """(window_us, t_xfer_us, raw budget) of the most recent window profile on this context."""
    w, t, b = C.c_double(), C.c_double(), C.c_int()
    _check(load().spm_get_profile(ctx, C.byref(w), C.byref(t), C.byref(b)), ctx)
    return w.value, t.value, b.value


def spm_measure_read_bandwidth(ctx, nbytes, reps=5) -> float:
    g = C.c_double()
    _check(load().spm_measure_read_bandwidth(ctx, nbytes, reps, C.byref(g)), ctx)
    return g.value


def spm_time_ffn_kernel(ctx, first_layer, x_norm, ids: np.ndarray, w, chained=True):
    """(us per launch by one event pair around all launches, mean in-kernel window in us)."""
    ids = np.ascontiguousarray(ids, np.int32)
    us, win = C.c_double(), C.c_double()
    _check(load().spm_time_ffn_kernel(ctx, first_layer, _ptr(x_norm), _ptr(ids), _ptr(w), ids.shape[0], int(chained),
                                      C.byref(us), C.byref(win)), ctx)
    return us.value, win.value


def spm_set_event_log_limit(ctx, max_events):
    _check(load().spm_set_event_log_limit(ctx, max_events), ctx)


def spm_set_device_wait_limit_us(ctx, us):
    _check(load().spm_set_device_wait_limit_us(ctx, us), ctx)


def spm_test_withhold_arrivals(ctx, count):
    _check(load().spm_test_withhold_arrivals(ctx, count), ctx)


def spm_cache_reset(ctx):
    _check(load().spm_cache_reset(ctx), ctx)


def spm_check_invariants(ctx, with_device=True):
    _check(load().spm_check_invariants(ctx, int(with_device)), ctx)


def spm_cache_export(ctx) -> np.ndarray:
    """The expert cache's checkpoint words (int64)."""
    n = C.c_size_t()
    _check(load().spm_cache_export(ctx, None, 0, C.byref(n)), ctx)
    out = np.empty(n.value, np.int64)
    _check(load().spm_cache_export(ctx, _ptr(out), out.size, C.byref(n)), ctx)
    return out


def spm_cache_import(ctx, state):
    state = np.ascontiguousarray(state, np.int64)
    _check(load().spm_cache_import(ctx, _ptr(state), state.size), ctx)


def spm_reset_stats(ctx):
    _check(load().spm_reset_stats(ctx), ctx)


def spm_get_stats(ctx) -> dict:
    st = Stats()
    _check(load().spm_get_stats(ctx, C.byref(st)), ctx)
    return st.as_dict()


def spm_get_layer_times(ctx, n_layers):
    stall = np.zeros(n_layers, np.float64)
    ffn = np.zeros(n_layers, np.float64)
    steps = C.c_uint64()
    _check(load().spm_get_layer_times(ctx, _ptr(stall), _ptr(ffn), C.byref(steps)), ctx)
    return stall, ffn, steps.value


def _events(fn, handle):
    n = C.c_size_t()
    _check(fn(handle, None, 0, C.byref(n)))
    buf = (Event * max(n.value, 1))()
    _check(fn(handle, C.cast(buf, _P), n.value, C.byref(n)))
    return [(e.step, e.layer, EVENT_NAMES[e.kind], e.expert, e.slot) for e in buf[:n.value]]


def spm_get_events(ctx):
    return _events(load().spm_get_events, ctx)


def spm_get_slot_table(ctx, layer, slots) -> np.ndarray:
    out = np.empty(slots, np.int32)
    _check(load().spm_get_slot_table(ctx, layer, _ptr(out)), ctx)
    return out


def spm_synchronize(ctx):
    _check(load().spm_synchronize(ctx), ctx)


def spm_ffn_noalloc(cfg: ModelCfg, blobs, n_blobs, which, w, x_norm, h_inout, stream=None, wait_and_check=False):
    """Expert FFN of one token for callers that may not allocate (see include/spm.h): no context,
    no arena; the partial rows go to a fixed array inside the library. `which` is a host list of
    blob indices, everything else is device memory; `stream` a raw cudaStream_t (None = default)."""
    which = np.ascontiguousarray(which, np.int32)
    _check(load().spm_ffn_noalloc(C.byref(cfg), _ptr(blobs), n_blobs, _ptr(which), _ptr(w), len(which),
                                  _ptr(x_norm), _ptr(h_inout), stream, int(wait_and_check)))


def spm_plan_grouped_chunks(n_units, n_dt, grid):
    """chunks[count][3] = unit, dt0, dt1 of the grouped tensor-core kernel's phase-2 chunk list."""
    cap = n_units * n_dt
    chunks = np.zeros((cap, 3), np.int32)
    count = C.c_size_t()
    _check(load().spm_plan_grouped_chunks(n_units, n_dt, grid, _ptr(chunks), cap, C.byref(count)))
    return chunks[:count.value]


def spm_host_alloc(nbytes: int) -> int:
    out = _P()
    _check(load().spm_host_alloc(nbytes, C.byref(out)))
    return out.value


def spm_host_free(ptr):
    _check(load().spm_host_free(ptr))


# ---- host-only slot-table simulator -----------------------------------------
class Sim:
    """Host-only slot table (spm_sim_*): drives the library's cache policy without a GPU."""

    def __init__(self, n_layers, n_experts, slots, plain_lru=False):
        out = _P()
        _check(load().spm_sim_create(n_layers, n_experts, slots, int(plain_lru), C.byref(out)))
        self.h, self.n, self.S = out.value, n_experts, slots

    def close(self):
        if self.h:
            load().spm_sim_destroy(self.h)
            self.h = None

    __del__ = close

    def demand(self, layer, need):
        need = np.ascontiguousarray(list(need), np.int32)
        outs = [np.empty(self.n, np.int32) for _ in range(4)]
        cnt, waves = C.c_int(), C.c_int()
        _check(load().spm_sim_demand(self.h, layer, _ptr(need), len(need), *[_ptr(o) for o in outs],
                                     C.byref(cnt), C.byref(waves)))
        res = [[] for _ in range(waves.value)]
        for i in range(cnt.value):
            res[outs[2][i]].append((int(outs[0][i]), int(outs[1][i]), bool(outs[3][i])))
        return res

    def plan(self, layer, ranking, budget, protect_all=False):
        ranking = np.ascontiguousarray(list(ranking), np.int32)
        sel, prot = np.empty(self.n, np.int32), np.empty(self.n, np.int32)
        ns, npr = C.c_int(), C.c_int()
        _check(load().spm_sim_plan(self.h, layer, _ptr(ranking), len(ranking), budget, int(protect_all),
                                   _ptr(sel), C.byref(ns), _ptr(prot), C.byref(npr)))
        return [int(e) for e in sel[:ns.value]], [int(e) for e in prot[:npr.value]]

    def prefetch(self, layer, ids, protect, drop_modulo=0):
        ids = np.ascontiguousarray(list(ids), np.int32)
        protect = np.ascontiguousarray(list(protect), np.int32)
        slots = np.full(max(len(ids), 1), -1, np.int32)
        issued = C.c_int()
        _check(load().spm_sim_prefetch(self.h, layer, _ptr(ids), len(ids), _ptr(protect), len(protect),
                                       drop_modulo, _ptr(slots), C.byref(issued)))
        return [(int(e), int(s)) for e, s in zip(ids, slots[:len(ids)]) if s >= 0]

    def plan_only(self, layer, ids):
        ids = np.ascontiguousarray(list(ids), np.int32)
        _check(load().spm_sim_plan_only(self.h, layer, _ptr(ids), len(ids)))

    def end_step(self):
        _check(load().spm_sim_end_step(self.h))

    def events(self):
        return _events(load().spm_sim_events, self.h)

    def stats(self) -> dict:
        st = Stats()
        _check(load().spm_sim_stats(self.h, C.byref(st)))
        return st.as_dict()

    def slot_table(self, layer):
        out = np.empty(self.S, np.int32)
        _check(load().spm_sim_slot_table(self.h, layer, _ptr(out)))
        return [int(e) for e in out]

    def check(self):
        _check(load().spm_sim_check(self.h))

    def export_state(self) -> np.ndarray:
        n = C.c_size_t()
        _check(load().spm_sim_export(self.h, None, 0, C.byref(n)))
        out = np.empty(n.value, np.int64)
        _check(load().spm_sim_export(self.h, _ptr(out), out.size, C.byref(n)))
        return out

    def import_state(self, state):
        state = np.ascontiguousarray(state, np.int64)
        _check(load().spm_sim_import(self.h, _ptr(state), state.size))
