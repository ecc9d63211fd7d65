"""The five workload configurations at their full sizes, in the launch configuration bench.py times.

For every head: routing (C_struct, label, p_v, p_s) and the index lists against the oracle's steps O1-O6
(all pooled-estimation heads included).  Attention: sampled query blocks against the oracle's exact
attention over the GPU's own lists - per head block 0, block N_b - 1, the block with the longest list and
random ones stratified over the four quartiles of m:
    L32k   every head, 32 blocks (seed 0; 16 for seeds 1 and 2)
    L128k  every head, 16 blocks
    Q256k  every head, 32 blocks
    L512k  every head, 64 blocks
With CRISP_TEST_FULL=1 L32k is checked on all of its 256 query blocks per head.
The oracle runs in a pool of worker processes (tests/parity_utils.py); the whole file takes about five minutes
on a 16-core host.
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


def _one_head_per_group_and_class(w):
    """The first head of every head class inside every KV group."""
    seen, heads = set(), []
    for h, cls in enumerate(w.head_classes):
        key = (h // w.group, cls)
        if key not in seen:
            seen.add(key)
            heads.append(h)
    return heads


def _block_fetcher(layer):
    def fetch(h, m):
        return layer.o[m * 128:(m + 1) * 128, h].float().cpu().numpy()
    return fetch


def _config_check(w, attention_heads, blocks_default, blocks_full, dense_blocks=4, report=None, band_limit=None):
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    name = w.name + (f" seed {w.seed}" if w.seed else "")
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
    lens = np.diff(g["row_ptr"], axis=1)
    per_head = blocks_full if FULL else blocks_default
    heads = list(range(hq)) if (FULL or attention_heads == "all") else _one_head_per_group_and_class(w)
    with pu.OraclePool(p, qc, kc, vc, g) as pool:
        # routing and lists: every head
        res, labels, excused = pool.heads(g, list(range(hq)), band_limit=band_limit or pu.BAND_LIMIT)
        t_lists = time.time() - t0
        samples = []
        for h in heads:
            longest = int(np.argmax(lens[h]))
            samples += [s for s in pu.sample_blocks(nb, hq, per_head, seed=h, always=(longest,)) if s[0] == h]
        rel, mab, blocks = pool.attention(g, samples, _block_fetcher(layer), lse=g["lse"])
        # the dense kernel on the same inputs: the last block of two heads and two blocks inside
        layer.dense_prefill(q, k, v)
        layer.poll()
        torch.cuda.synchronize()
        lse_dense = layer.lse.cpu().numpy()
        picks = [(heads[0], nb - 1), (heads[-1], nb - 1), (heads[len(heads) // 2], nb // 2), (heads[0], 0),
                 (heads[-1], nb // 3), (heads[1 % len(heads)], 1)][:dense_blocks]
        drel, dmab, dblocks = pool.attention(g, picks, _block_fetcher(layer), lse=lse_dense, dense=True)
    n_vs = int((g["pattern"] == orc.VS).sum())
    frac = nnz / (hq * nb * (nb + 1) // 2)
    line = (f"{name}: lists of all {hq} heads ({n_vs} VS, {hq - n_vs} PE) match; excused labels {labels}; excused "
            f"blocks: {excused}; block fraction {frac:.3f}; attention on {len(samples)} query blocks "
            f"({per_head} per head on {len(heads)} heads, {blocks} key blocks): rel-L2 {rel:.2e}, max-abs {mab:.2e}; "
            f"dense kernel on {len(picks)} query blocks ({dblocks} key blocks): rel-L2 {drel:.2e}, max-abs {dmab:.2e}; "
            f"{t_lists:.0f} s lists + {time.time() - t0 - t_lists:.0f} s attention")
    print(line)
    if report is not None:
        report(line)
    return layer, g, (q, k, v), (qc, kc, vc), res


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_config_L32k(seed, parity_report):
    w = synth.CONFIGS["L32k"].with_(seed=seed)
    _config_check(w, "all", blocks_default=32 if seed == 0 else 16, blocks_full=256, report=parity_report)


def test_config_L128k_alpha_sweep_and_gamma_selector(parity_report):
    pu = _pu()
    w = synth.CONFIGS["L128k"]
    layer, g, (q, k, v), (qc, kc, vc), res = _config_check(w, "all", blocks_default=16, blocks_full=64,
                                                            report=parity_report)
    hq, nb = w.n_q_heads, w.n_blocks
    vs_heads = [h for h in range(hq) if g["pattern"][h] == orc.VS]
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
        exc = pu.check_lists(g2, res2, p2, heads=vs_heads, band_limit=pu.BAND_LIMIT)
        rows_vs = sum(int(np.diff(g2["row_ptr"][h]).sum()) for h in vs_heads)
        nnz_by[label] = rows_vs
        line = f"L128k {label}: lists of all {len(vs_heads)} VS heads match; excused blocks: {exc}; listed blocks {rows_vs}"
        print(line)
        parity_report(line)
    base = sum(int(np.diff(g["row_ptr"][h]).sum()) for h in vs_heads)
    assert nnz_by["alpha=2.0"] <= base <= nnz_by["alpha=0.5"]


def test_config_Q256k(parity_report):
    # the sink-dominated heads have a flat background: ~8 % of their blocks lie within 0.1 % of alpha * mu
    _config_check(synth.CONFIGS["Q256k"], "all", blocks_default=32, blocks_full=64, report=parity_report,
                  band_limit=0.10)


def test_config_L512k(parity_report):
    _config_check(synth.CONFIGS["L512k"], "all", blocks_default=64, blocks_full=64, report=parity_report)


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
    # head 1 is a diffuse head forced to Vertical-Slash: its block scores are flat, so a third of them lie in
    # the 1e-3 band around alpha * mu
    excused = pu.check_lists(g, res, p, band_limit=1.0)
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
