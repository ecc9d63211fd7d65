"""The five workload configurations at their full sizes, in the launch configuration bench.py times.

Routing (C_struct, labels, p_v, p_s) is checked for every head; the index lists for every VS head and a
subset of the PE heads (all of them with CRISP_TEST_FULL=1); attention on sampled query blocks against
the oracle's exact attention over the GPU's own lists (64 per head at 512k with CRISP_TEST_FULL=1,
fewer by default so that the suite stays within a few minutes of host time).
"""
import os
import time

import numpy as np
import pytest
import torch

from oracle import crisp_oracle as orc
from workloads import synth

pytestmark = pytest.mark.gpu
FULL = os.environ.get("CRISP_TEST_FULL", "0") == "1"


def _pu():
    from tests import parity_utils
    return parity_utils


def _oracle_heads(qc, kc, p, heads, pu):
    hq, hkv = p.n_q_heads, p.n_kv_heads
    kw = pu.oracle_kwargs(p)
    out = [None] * hq
    for h in heads:
        out[h] = orc.head_pipeline(qc[:, h].float().numpy(), kc[:, orc.kv_head(h, hq, hkv)].float().numpy(), **kw)
    return out


def _route_only(qc, kc, p, h):
    """Oracle steps O1-O3 of one head (cheap at any size)."""
    hq, hkv = p.n_q_heads, p.n_kv_heads
    a = orc.proxy_attention(qc[:, h].float().numpy(), kc[:, orc.kv_head(h, hq, hkv)].float().numpy(), p.block)
    c = orc.c_struct(a, p.sink_tokens, p.local_tokens)
    p_v, p_s = orc.block_scores(a, p.block)
    return dict(c_struct=c, pattern=orc.route(c, p.tau), p_v=p_v, p_s=p_s)


def _config_check(name, pe_heads_default, blocks_default, blocks_full, dense_blocks=2):
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    w = synth.CONFIGS[name]
    p = pu.params_of(w)
    t0 = time.time()
    q, k, v = synth.make_qkv(w, device="cuda")
    layer = crisp.CrispLayer(p, with_lse=True)
    layer.forward(q, k, v)
    layer.poll()
    torch.cuda.synchronize()
    nnz = int(layer.nnz.item())
    g = dict(c_struct=layer.c_struct.cpu().numpy(), pattern=layer.pattern.cpu().numpy(),
             p_v=layer.p_v.cpu().numpy(), p_s=layer.p_s.cpu().numpy(), row_ptr=layer.row_ptr.cpu().numpy(),
             col_idx=layer.col_idx[:nnz].cpu().numpy(), nnz=nnz, o=None, lse=layer.lse.cpu().numpy())
    qc, kc, vc = q.cpu(), k.cpu(), v.cpu()
    hq, nb = w.n_q_heads, w.n_blocks
    # routing for every head
    labels = 0
    route_res = [_route_only(qc, kc, p, h) for h in range(hq)]
    labels = pu.check_route(g, route_res, p)
    # lists: every VS head, some PE heads
    vs_heads = [h for h in range(hq) if route_res[h]["pattern"] == orc.VS]
    pe_heads = [h for h in range(hq) if route_res[h]["pattern"] == orc.PE]
    if not FULL:
        pe_heads = pe_heads[:pe_heads_default]
    res = _oracle_heads(qc, kc, p, vs_heads + pe_heads, pu)
    excused = pu.check_lists(g, res, p, heads=vs_heads + pe_heads)
    # attention on sampled query blocks: the output tensor is pulled block by block
    per_head = blocks_full if FULL else blocks_default
    lens = np.diff(g["row_ptr"], axis=1)
    heads = range(hq) if FULL else sorted(set(vs_heads[:2] + pe_heads[:2] + [hq - 1]))
    samples = []
    for h in heads:
        longest = int(np.argmax(lens[h]))
        samples += [s for s in pu.sample_blocks(nb, hq, per_head, seed=h, always=(longest,)) if s[0] == h]
    o_host = {}
    for h, m in samples:
        o_host[(h, m)] = layer.o[m * 128:(m + 1) * 128, h].float().cpu().numpy()

    class _O:
        def __getitem__(self, idx):
            rows, h = idx
            return o_host[(h, rows.start // 128)]
    g["o"] = _O()
    rel, mab = pu.check_attention(g, qc, kc, vc, p, samples)
    # the dense kernel on the same inputs
    layer.dense_prefill(q, k, v)
    layer.poll()
    torch.cuda.synchronize()
    g["lse_dense"] = layer.lse.cpu().numpy()
    dense_samples = [(h, m) for h, m in samples if m in (0, nb - 1)][:dense_blocks * 2]
    for h, m in dense_samples:
        o_host[(h, m)] = layer.o[m * 128:(m + 1) * 128, h].float().cpu().numpy()
    g["o_dense"] = g["o"]
    pu.check_attention(g, qc, kc, vc, p, dense_samples, key="o_dense", dense=True)
    frac = nnz / (hq * nb * (nb + 1) // 2)
    print(f"{name}: VS heads {len(vs_heads)}, PE heads checked {len(pe_heads)}, excused labels {labels}, "
          f"excused blocks {excused}, block fraction {frac:.3f}, {len(samples)} sampled blocks, "
          f"rel-L2 {rel:.2e}, max-abs {mab:.2e}, {time.time() - t0:.0f} s")
    return layer, g, (q, k, v), (qc, kc, vc), res


def test_config_L32k():
    _config_check("L32k", pe_heads_default=4, blocks_default=6, blocks_full=256)


def test_config_L128k_alpha_sweep_and_gamma_selector():
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    layer, g, (q, k, v), (qc, kc, vc), res = _config_check("L128k", pe_heads_default=2, blocks_default=4,
                                                            blocks_full=64)
    w = synth.CONFIGS["L128k"]
    hq, nb = w.n_q_heads, w.n_blocks
    vs_heads = [h for h in range(hq) if g["pattern"][h] == orc.VS][: (hq if FULL else 4)]
    nnz_by = {}
    for label, over in (("alpha=0.5", dict(alpha=0.5)), ("alpha=2.0", dict(alpha=2.0)),
                        ("gamma=0.95", dict(selector=1))):
        p2 = pu.params_of(w, **over)
        layer.p = p2
        layer.select(q, k)
        layer.poll()
        torch.cuda.synchronize()
        nnz = int(layer.nnz.item())
        g2 = dict(g, row_ptr=layer.row_ptr.cpu().numpy(), col_idx=layer.col_idx[:nnz].cpu().numpy(), nnz=nnz)
        res2 = [None] * hq
        for h in vs_heads:
            r = res[h]
            if over.get("selector") == 1:
                s_v, kv_, raw_v = orc.select_gamma(r["p_v"], p2.gamma, p2.k_min_blocks)
                s_s, ks_, raw_s = orc.select_gamma(r["p_s"], p2.gamma, p2.k_min_blocks)
            else:
                s_v, kv_, raw_v = orc.select_noise_floor(r["p_v"], p2.alpha, p2.k_min_blocks)
                s_s, ks_, raw_s = orc.select_noise_floor(r["p_s"], p2.alpha, p2.k_min_blocks)
            res2[h] = dict(r, s_v=s_v, s_s=s_s, k_v=kv_, k_s=ks_, raw_v=raw_v, raw_s=raw_s,
                           cols=orc.expand_vs(s_v, s_s, nb))
        exc = pu.check_lists(g2, res2, p2, heads=vs_heads)
        rows_vs = sum(int(np.diff(g2["row_ptr"][h]).sum()) for h in vs_heads)
        nnz_by[label] = rows_vs
        print(f"L128k {label}: excused blocks {exc}, listed blocks on {len(vs_heads)} VS heads {rows_vs}")
    base = sum(int(np.diff(g["row_ptr"][h]).sum()) for h in vs_heads)
    assert nnz_by["alpha=2.0"] <= base <= nnz_by["alpha=0.5"]


def test_config_Q256k():
    _config_check("Q256k", pe_heads_default=1, blocks_default=3, blocks_full=64)


def test_config_L512k():
    _config_check("L512k", pe_heads_default=1, blocks_default=3, blocks_full=64)


def test_maximum_block_count_one_million_tokens():
    """N_b = 8192 (the selection kernels' limit): 1,048,576 tokens, 2 query heads on 1 KV head."""
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    from paper_2609_01925_b200 import binding as B
    n = 8192 * 128
    w = synth.llama_shaped("M1M", n, 64).with_(n_q_heads=2, n_kv_heads=1, head_classes=("conc", "diffuse"))
    p = pu.params_of(w, force_pattern=1)
    q, k, v = synth.make_qkv(w, device="cuda", chunk_tokens=65536)
    layer = crisp.CrispLayer(p, with_lse=True)
    layer.forward(q, k, v)
    layer.poll()
    torch.cuda.synchronize()
    nnz = int(layer.nnz.item())
    g = dict(c_struct=layer.c_struct.cpu().numpy(), pattern=layer.pattern.cpu().numpy(),
             p_v=layer.p_v.cpu().numpy(), p_s=layer.p_s.cpu().numpy(), row_ptr=layer.row_ptr.cpu().numpy(),
             col_idx=layer.col_idx[:nnz].cpu().numpy(), nnz=nnz, lse=layer.lse.cpu().numpy())
    qc, kc, vc = q.cpu(), k.cpu(), v.cpu()
    res = _oracle_heads(qc, kc, p, [0, 1], pu)
    pu.check_route(g, res, p)
    excused = pu.check_lists(g, res, p)
    nb = w.n_blocks
    samples = [(0, 0), (0, nb - 1), (0, 5000), (1, nb - 1), (1, 1234)]
    o_host = {(h, m): layer.o[m * 128:(m + 1) * 128, h].float().cpu().numpy() for h, m in samples}

    class _O:
        def __getitem__(self, idx):
            rows, h = idx
            return o_host[(h, rows.start // 128)]
    g["o"] = _O()
    rel, mab = pu.check_attention(g, qc, kc, vc, p, samples)
    print(f"M1M: nnz {nnz}, excused blocks {excused}, rel-L2 {rel:.2e}, max-abs {mab:.2e}")
    # one block more is refused on the host
    p2 = crisp.make_params(n + 128, 2, 1)
    assert B.load().crisp_select(__import__("ctypes").byref(p2), 1, 1, 1, 1, 1, 1, 1 << 40, 1, 1, 1, 1, None) \
        in (B.ERR_UNSUPPORTED, B.ERR_INVALID_ARG, B.ERR_WORKSPACE)
