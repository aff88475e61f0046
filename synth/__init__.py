"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path.

This package holds input generation only: no router, adapter, expert or cache
arithmetic lives here.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    ModelCfg,
    TAG_ADAPTER_A,
    TAG_ADAPTER_B,
    TAG_DOWN,
    TAG_EMB,
    TAG_GATE,
    TAG_ROUTER,
    TAG_UP,
    adapter_a,
    adapter_b,
    dequantize_q4,
    embedding_rows,
    expert_matrices,
    expert_q4,
    quantize_q4,
    get_config,
    normal_table,
    router_w,
    synth_normal,
    zipf_probs,
    zipf_tokens,
)
