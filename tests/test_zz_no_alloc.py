"""spm_ffn_noalloc: the expert FFN for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is forbidden (a serving loop with a frozen memory
map, a process whose device memory belongs to another allocator), so they can create neither an
arena nor an spm_ctx. The entry point tested here needs neither: its scratch is a fixed array inside
the library. This file checks, through the C ABI, that it gives the same result as spm_moe_ffn
and as the CPU oracle's plain definition of the expert layer, on two calls in a row (the second
call finds the first call's leftovers in the shared array).
It is collected last on purpose, so a run that stops at the first failure has already run the rest.
"""
import numpy as np
import pytest
import torch

import synth
from helpers import SynthWeights
from oracle import ref_math as M

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "qw_small"])
def test_noalloc_matches_moe_ffn_twice_in_a_row(name):
    from paper_2607_24787_b200 import binding as B
    from paper_2607_24787_b200.build import build
    from paper_2607_24787_b200.model import pack_experts
    from paper_2607_24787_b200.synth_model import build_from_synth
    build()
    cfg = {"tiny": synth.get_config("tiny"),
           "qw_small": synth.get_config("qwen3", n_layers=2, n_experts=24, inter=96, slots=24, budget=0)}[name]
    m = build_from_synth(cfg, slots=cfg.n_experts, budget=0)          # the existing entry point, all experts resident
    layer = 1
    g, u, d = synth.expert_matrices(cfg, layer, range(cfg.n_experts), device="cuda")
    blobs = pack_experts(g, u, d).contiguous()                         # device copy of the layer's packed experts
    rng = np.random.default_rng(11)
    torch.manual_seed(1234)                                            # same inputs on every run
    wts = SynthWeights(cfg)
    tol = 1e-5 if cfg.dtype == "fp32" else 1e-4
    stream = torch.cuda.Stream()
    for call in range(2):
        ids = np.sort(rng.permutation(cfg.n_experts)[:cfg.top_k]).astype(np.int32)
        x = torch.randn(1, cfg.hidden, device="cuda")
        w = torch.rand(1, cfg.top_k, device="cuda")
        h0 = torch.randn(1, cfg.hidden, device="cuda")
        h_ref, h_new = h0.clone(), h0.clone()
        torch.cuda.synchronize()
        m.moe_ffn(layer, x, ids[None], w, h_ref)
        m.synchronize()
        B.spm_ffn_noalloc(m.cfg, blobs, cfg.n_experts, ids, w, x, h_new, stream.cuda_stream, wait_and_check=True)
        a, b = h_new.cpu().numpy().astype(np.float64), h_ref.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(a - b)) / np.max(np.abs(b)) < tol, call
        assert not np.array_equal(b, h0.cpu().numpy())                 # the FFN did change h
        # ... and against the oracle's definition y = sum_k w_k FFN_k(x), computed from the same weights
        y = M.moe_ffn(x[0].cpu().numpy().astype(np.float64), ids, w[0].cpu().numpy().astype(np.float64),
                      lambda e: wts.expert(layer, e))
        h064 = h0[0].cpu().numpy().astype(np.float64)
        assert M.rel_linf(a[0], h064 + y) < tol, call
        # the update itself, y = h_new - h0: h is kept in fp32, so the difference carries its rounding (2^-24 of max|h|)
        assert M.rel_linf(a[0] - h064, y) < tol + 2.0 ** -23 * np.max(np.abs(h064)) / np.max(np.abs(y)), call
    # sizes beyond the built-in array are refused with a message, nothing is launched
    big = B.make_cfg(1, 4096, 8, 64, 2, 0, 4, B.DTYPE_BF16)
    with pytest.raises(B.SpmError) as e:
        B.spm_ffn_noalloc(big, blobs, 8, [0, 1], w, x, h_new, stream.cuda_stream)
    assert e.value.code == -2 and "scratch" in str(e.value)
    with pytest.raises(B.SpmError):
        B.spm_ffn_noalloc(m.cfg, blobs, cfg.n_experts, [cfg.n_experts], w, x, h_new, stream.cuda_stream)
    # a misaligned view (here: a row that starts 4 bytes into a buffer) is refused, not launched
    pad = torch.zeros(cfg.hidden + 4, device="cuda")
    with pytest.raises(B.SpmError) as e:
        B.spm_ffn_noalloc(m.cfg, blobs, cfg.n_experts, ids, w, pad[1:cfg.hidden + 1], h_new, stream.cuda_stream)
    assert e.value.code == -1 and "aligned" in str(e.value)
    m.close()
