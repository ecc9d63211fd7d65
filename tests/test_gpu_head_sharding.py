"""Head-sharded layout on the GPU: the KV groups of one layer are split as two ranks would hold them, both shards
run one after the other on this device through the unchanged C-ABI calls (they are independent: nothing waits on
anything), and every output of a shard equals the single-rank output of the same heads bit for bit."""
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import sharding
from workloads import synth

pytestmark = pytest.mark.gpu


def _run(w, q, k, v):
    p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens,
                          local_tokens=w.local_tokens, k_min_blocks=w.k_min_blocks, tau=w.tau, alpha=w.alpha,
                          gamma=w.gamma)
    layer = crisp.CrispLayer(p, with_lse=True)
    layer.forward(q, k, v)
    layer.poll()
    torch.cuda.synchronize()
    return layer


def test_shards_reproduce_the_single_rank_outputs():
    w = synth.llama_shaped("shard-test", 4096, 16).with_(n_q_heads=16, n_kv_heads=4,
                                                          head_classes=("conc", "diffuse") * 8)
    q, k, v = synth.make_qkv(w, device="cuda")
    full = _run(w, q, k, v)
    nb = w.n_blocks
    full_rp = full.row_ptr.cpu()
    world = 2
    for rank in range(world):
        groups = sharding.kv_groups_of_rank(w.n_kv_heads, rank, world)
        heads = sharding.q_heads_of_groups(groups, w.group)
        qs, ks, vs = synth.make_qkv_kv_groups(w, groups, device="cuda")
        assert torch.equal(qs, q[:, heads]) and torch.equal(ks, k[:, groups]) and torch.equal(vs, v[:, groups])
        ws = w.with_(n_q_heads=len(heads), n_kv_heads=len(groups), head_classes=tuple(w.head_classes[h] for h in heads))
        part = _run(ws, qs, ks, vs)
        assert torch.equal(part.o, full.o[:, heads])
        assert torch.equal(part.lse, full.lse[heads])
        assert torch.equal(part.pattern, full.pattern[heads])
        assert torch.equal(part.c_struct, full.c_struct[heads])
        assert torch.equal(part.p_v, full.p_v[heads]) and torch.equal(part.p_s, full.p_s[heads])
        rp = part.row_ptr.cpu()
        for j, h in enumerate(heads):
            a = part.col_idx[int(rp[j, 0]):int(rp[j, nb])]
            b = full.col_idx[int(full_rp[h, 0]):int(full_rp[h, nb])]
            assert torch.equal(a, b)
            assert torch.equal(rp[j] - rp[j, 0], full_rp[h] - full_rp[h, 0])
