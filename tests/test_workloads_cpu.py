"""The synthetic generator: determinism, shapes, planted structure (no method arithmetic here)."""
import numpy as np
import torch

from workloads import synth


def test_generator_is_deterministic_and_chunk_independent():
    w = synth.tiny(n=1024)
    q1, k1, v1 = synth.make_qkv(w, chunk_tokens=1024)
    q2, k2, v2 = synth.make_qkv(w, chunk_tokens=200)
    assert torch.equal(q1, q2) and torch.equal(k1, k2) and torch.equal(v1, v2)
    q3, _, _ = synth.make_qkv(w.with_(seed=1))
    assert not torch.equal(q1, q3)


def test_shapes_and_dtypes_of_every_config():
    for name, w in synth.CONFIGS.items():
        assert w.seq_len % 128 == 0 and w.n_q_heads % w.n_kv_heads == 0
        assert len(w.head_classes) == w.n_q_heads
    w = synth.CONFIGS["Tiny"]
    q, k, v = synth.make_qkv(w)
    assert q.shape == (4096, 4, 128) and k.shape == v.shape == (4096, 1, 128)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16


def test_normal_generator_moments():
    x = synth.normal(0, 7, torch.arange(1 << 18)).double()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    assert abs((x ** 4).mean().item() - 3.0) < 0.1


def test_planted_structure_is_where_the_recipe_says():
    w = synth.llama_shaped("t", 4096, 8).with_(n_q_heads=4, n_kv_heads=1,
                                              head_classes=("conc", "diffuse", "conc", "diffuse"))
    q, k, v = synth.make_qkv(w)
    u = torch.zeros(128); u[52:64] = 1; u[116:128] = 1
    proj = (k[:, 0].float() @ u) / 24.0          # mean of the U components
    cols = synth.planted_columns(w, 0)
    assert all(128 <= c < 4096 - 128 for c in cols)
    assert torch.all(proj[:4] > 7.5)
    assert torch.all(proj[cols] > 3.5)
    mask = torch.ones(4096, dtype=torch.bool); mask[:4] = False; mask[cols] = False
    assert proj[mask].abs().max() < 1e-6
    # slash lines: the W part of q_i . k_j peaks at i - j in the planted offsets
    wm = torch.zeros(128); wm[0:32] = 1; wm[64:96] = 1
    i = 3000
    logits = ((q[i, 0].float() * wm) @ (k[:, 0].float() * wm).T)[: i + 1]
    offsets = i - torch.arange(i + 1)
    far = (offsets > 300) & ((offsets - 1056).abs() > 64)      # away from every planted line
    for delta in (1, 96, 1056):
        near = (offsets - delta).abs() <= 3
        assert logits[near].max() > logits[far].max()
    # diffuse heads carry no planted component
    assert (q[:, 1].float() * (u + wm)).abs().max() == 0
