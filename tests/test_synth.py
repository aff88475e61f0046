"""Pins for the synthetic input generators (CPU only)."""
import numpy as np
import torch

import synth


def test_zipf_closed_forms():
    # P(id 0) = 1 / H_{V,1.1}; cumulative mass of the 16 most frequent ids
    for V, p0, top16 in ((1024, 0.17906, 0.542), (129280, 0.13329, 0.404), (151936, 0.13242, 0.401)):
        p = synth.zipf_probs(V)
        assert abs(p[0] - p0) < 5e-6 and abs(p[:16].sum() - top16) < 1e-3
        assert abs(p.sum() - 1.0) < 1e-12 and np.all(np.diff(p) < 0)


def test_zipf_tokens_deterministic_and_distributed():
    cfg = synth.get_config("tiny")
    a = synth.zipf_tokens(cfg, steps=4000)
    b = synth.zipf_tokens(cfg, steps=4000)
    assert a.shape == (4000, 1) and np.array_equal(a, b)
    assert a.min() >= 0 and a.max() < cfg.vocab
    assert abs((a == 0).mean() - 0.17906) < 0.02
    c = synth.zipf_tokens(cfg, steps=4000, stream=1)
    assert not np.array_equal(a, c)
    bt = synth.zipf_tokens(synth.get_config("batched"), steps=3)
    assert bt.shape == (3, 64)


def test_counter_based_weights():
    cfg = synth.get_config("tiny")
    g, u, d = synth.expert_matrices(cfg, 1, [0, 3, 15])
    g3, u3, d3 = synth.expert_matrices(cfg, 1, [3])
    assert torch.equal(g[1], g3[0]) and torch.equal(u[1], u3[0]) and torch.equal(d[1], d3[0])
    assert g.shape == (3, cfg.inter, cfg.hidden) and d.shape == (3, cfg.hidden, cfg.inter)
    assert g.dtype == torch.float32
    assert abs(g.std().item() - 0.02) < 5e-4 and abs(g.mean().item()) < 5e-4
    assert not torch.equal(g[0], u[0]) and not torch.equal(g[0], g[1])
    big = synth.get_config("dsvl2")
    w = synth.router_w(big, 2)
    assert w.dtype == torch.bfloat16 and w.shape == (64, 1280)
    assert abs(w.float().std().item() - 0.02) < 5e-4
    e = synth.embedding_rows(big, [5, 0, 5])
    assert e.dtype == torch.float32 and torch.equal(e[0], e[2]) and not torch.equal(e[0], e[1])
    assert abs(e.std().item() - 1.0) < 0.05
    # stored in bf16: every value survives a bf16 round trip
    assert torch.equal(e, e.to(torch.bfloat16).to(torch.float32))


def test_config_table():
    q = synth.get_config("qwen3")
    assert q.expert_bytes == 9437184 and q.n_layers * q.n_experts * q.expert_bytes == 57982058496
    assert synth.get_config("dsvl2").expert_bytes == 6881280
    assert synth.get_config("tiny").expert_bytes == 393216


def test_q4_quantiser_and_packing():
    w = torch.randn(3, 5, 96) * 0.02
    w[0, 0, :32] = 0.0                                   # an all-zero group keeps scale 1, codes 8
    q, s = synth.quantize_q4(w)
    assert q.dtype == torch.uint8 and q.min() >= 1 and q.max() <= 15 and s.dtype == torch.float16
    assert s.shape == (3, 5, 3) and torch.all(q[0, 0, :32] == 8) and s[0, 0, 0] == 1
    deq = synth.dequantize_q4(q, s)
    err = (deq - w).abs().reshape(3, 5, 3, 32).amax(-1)
    assert torch.all(err <= s.float() * 0.5 + 1e-7)                       # round to nearest code
    assert torch.equal(deq, (q.double() - 8).mul(s.double().repeat_interleave(32, -1)).float())   # exact in fp32
    cfg = synth.get_config("dsvl2_q4")
    assert cfg.expert_bytes == 1935360                                    # the paper's 1.94 MB per expert
    assert synth.get_config("qwen3_q4").expert_bytes * 32 == synth.get_config("qwen3").expert_bytes * 9
    small = cfg.replace(n_layers=1, n_experts=3, inter=8)
    g, u, d = synth.expert_matrices(small, 0, [1])
    (gq, gs), (uq, us), (dq, dsc) = synth.expert_q4(small, 0, [1])
    assert torch.equal(g, synth.dequantize_q4(gq, gs)) and torch.equal(d, synth.dequantize_q4(dq, dsc).transpose(1, 2))
    from paper_2607_24787_b200.model import pack_experts_q4
    blob = pack_experts_q4((gq, gs), (uq, us), (dq, dsc))
    D = small.hidden
    assert blob.shape == (1, 8, 3, D // 2 + D // 16) and blob.numel() == small.expert_bytes
    nib = blob[0, 3, 2, :D // 2]
    assert torch.equal(torch.stack((nib & 15, nib >> 4), -1).reshape(-1), dq[0, 3])
    assert torch.equal(blob[0, 3, 2, D // 2:].view(torch.float16), dsc[0, 3])
