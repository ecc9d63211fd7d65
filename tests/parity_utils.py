"""Helpers shared by the GPU parity tests: run the C-ABI stages, run the oracle, compare.

Matching rule (per stage):
  * c_struct, p_v, p_s: floating point, rtol 2e-4 / atol 1e-7 (fp32 accumulation and the hardware
    exp2 approximation against an fp64 oracle).
  * routing labels: identical unless |C_struct - tau| <= 1e-3 * tau.
  * index lists: identical except for blocks whose score lies within 1e-3 (relative) of the deciding
    value (alpha * mu_d, or the value at the k_min / gamma cut).  With A the set of such blocks, the
    GPU list of every query block must lie between expand(S minus A) and expand(S union A).
    For the cumulative rules the entry right at the cut is also excused when the running sum passes
    within 1e-6 of gamma (fp32 scores against fp64).  The number of such blocks is returned.
  * attention output against the oracle's exact attention over the GPU's own lists:
    rel-L2 <= 1e-2 and max-abs <= 2e-2.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2609_01925_b200 as crisp
from oracle import crisp_oracle as orc

REL_BAND = 1e-3
MASS_BAND = 1e-6


def params_of(w, **over):
    kw = dict(sink_tokens=w.sink_tokens, local_tokens=w.local_tokens, k_min_blocks=w.k_min_blocks,
              tau=w.tau, alpha=w.alpha, gamma=w.gamma)
    kw.update(over)
    return crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, **kw)


def run_gpu(p, q, k, v, dense=False, with_lse=True, capacity=None):
    layer = crisp.CrispLayer(p, capacity=capacity, with_lse=with_lse)
    layer.route(q, k)
    layer.select(q, k)
    layer.poll()
    layer.sparse_prefill(q, k, v)
    layer.poll()
    torch.cuda.synchronize()
    out = dict(c_struct=layer.c_struct.cpu().numpy(), pattern=layer.pattern.cpu().numpy(),
               p_v=layer.p_v.cpu().numpy(), p_s=layer.p_s.cpu().numpy(),
               row_ptr=layer.row_ptr.cpu().numpy(), nnz=int(layer.nnz.item()),
               o=layer.o.float().cpu().numpy(), lse=layer.lse.cpu().numpy() if with_lse else None)
    out["col_idx"] = layer.col_idx[:out["nnz"]].cpu().numpy()
    if dense:
        layer.dense_prefill(q, k, v)
        layer.poll()
        torch.cuda.synchronize()
        out["o_dense"] = layer.o.float().cpu().numpy()
        out["lse_dense"] = layer.lse.cpu().numpy() if with_lse else None
    return out


def gpu_cols(g, h, m):
    rp = g["row_ptr"]
    return g["col_idx"][rp[h, m]:rp[h, m + 1]]


def oracle_kwargs(p):
    return dict(block=p.block, sink_tokens=p.sink_tokens, local_tokens=p.local_tokens, tau=p.tau,
                alpha=p.alpha, gamma=p.gamma, k_min_blocks=p.k_min_blocks, selector=p.selector,
                force_pattern=p.force_pattern,
                scale=(p.softmax_scale if p.softmax_scale > 0 else None))


def check_route(g, res, p, heads=None):
    """Returns the number of heads whose label was excused by the band around tau."""
    excused = 0
    heads = range(len(res)) if heads is None else heads
    for h in heads:
        r = res[h]
        np.testing.assert_allclose(g["c_struct"][h], r["c_struct"], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(g["p_v"][h], r["p_v"], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(g["p_s"][h], r["p_s"], rtol=2e-4, atol=1e-7)
        if g["pattern"][h] != r["pattern"]:
            assert abs(r["c_struct"] - p.tau) <= REL_BAND * p.tau, (h, r["c_struct"], g["c_struct"][h])
            excused += 1
    return excused


def _ambiguous_vs(pd, p, k_d, raw):
    """Blocks of one direction whose membership may legitimately differ."""
    nb = pd.shape[0]
    order = np.argsort(-pd, kind="stable")
    amb = np.zeros(nb, dtype=bool)
    if p.selector in (0, 2):
        mu = orc.noise_floor(pd)[1] if p.selector == 0 else float(np.median(pd[1:nb - 1]))
        thr = p.alpha * mu
        amb |= np.abs(pd - thr) <= REL_BAND * thr
    if p.selector == 1 and raw < nb:
        # the running sum may reach gamma one entry earlier or later when it passes within 1e-6 of it
        cs = np.cumsum(pd[order])
        if cs[raw - 1] - p.gamma <= MASS_BAND:
            amb[order[raw]] = True
        if raw >= 2 and p.gamma - cs[raw - 2] <= MASS_BAND:
            amb[order[raw - 1]] = True
    if p.selector == 1 or raw < p.k_min_blocks:
        if k_d < nb:
            cut = pd[order[k_d - 1]]
            amb |= np.abs(pd - cut) <= REL_BAND * cut
            nxt = pd[order[k_d]]
            amb |= np.abs(pd - nxt) <= REL_BAND * max(nxt, 1e-300)
    return amb


def _rows_to_matrix(cols_per_row, nb):
    m = np.zeros((nb, nb), dtype=bool)
    for r, c in enumerate(cols_per_row):
        m[r, c] = True
    return m


def gpu_matrix(g, h, nb):
    """Boolean [N_b, N_b] matrix of the GPU lists of head h; also checks order and bounds."""
    rp = g["row_ptr"][h]
    cols = g["col_idx"][rp[0]:rp[nb]].astype(np.int64)
    lens = np.diff(rp)
    rows = np.repeat(np.arange(nb), lens)
    assert lens.min() >= 1
    assert np.all(cols <= rows) and np.all(cols >= 0), (h, "column out of range")
    same_row = rows[1:] == rows[:-1]
    assert np.all(np.diff(cols)[same_row] > 0), (h, "not ascending/unique")
    first = rp[:-1] - rp[0]
    last = rp[1:] - rp[0] - 1
    assert np.all(cols[first] == 0) and np.all(cols[last] == np.arange(nb)), (h, "forced blocks missing")
    m = np.zeros((nb, nb), dtype=bool)
    m[rows, cols] = True
    return m


def check_lists(g, res, p, heads=None):
    """GPU lists vs oracle lists under the matching rule.  Returns the count of excused blocks."""
    nb = -(-p.seq_len // p.block)
    excused_total = 0
    heads = range(len(res)) if heads is None else heads
    for h in heads:
        r = res[h]
        if r is None or g["pattern"][h] != r["pattern"]:
            continue  # label excused by check_route; lists follow the other branch
        if nb <= 2:
            lo = hi = _rows_to_matrix(r["cols"], nb)
        elif r["pattern"] == orc.VS:
            amb_v = _ambiguous_vs(r["p_v"], p, r["k_v"], r["raw_v"])
            amb_s = _ambiguous_vs(r["p_s"], p, r["k_s"], r["raw_s"])
            sv = np.zeros(nb, bool); sv[r["s_v"]] = True
            ss = np.zeros(nb, bool); ss[r["s_s"]] = True
            lo = _rows_to_matrix(orc.expand_vs(np.nonzero(sv & ~amb_v)[0], np.nonzero(ss & ~amb_s)[0], nb), nb)
            hi = _rows_to_matrix(orc.expand_vs(np.nonzero(sv | amb_v)[0], np.nonzero(ss | amb_s)[0], nb), nb)
            excused_total += int(amb_v.sum() + amb_s.sum())
        else:
            flat = r["a_bar"] / r["a_bar"].sum()
            cut = r["pe_cut"]
            tri = np.tril(np.ones((nb, nb), bool))
            amb = (np.abs(flat - cut) <= REL_BAND * cut) & tri
            # mass band: the cumulative sum may pass within 1e-6 of gamma, moving the cut by one entry
            vals = np.where(tri, flat, -1.0).reshape(-1)
            order = np.argsort(-vals, kind="stable")[:tri.sum()]
            cs = np.cumsum(vals[order])
            kstar = int(r["pe_sel"].sum())
            if kstar < order.size and cs[kstar - 1] - p.gamma <= MASS_BAND:
                amb.reshape(-1)[order[kstar]] = True
            if kstar >= 2 and p.gamma - cs[kstar - 2] <= MASS_BAND:
                amb.reshape(-1)[order[kstar - 1]] = True
            lo = _rows_to_matrix(orc.expand_pe(r["pe_sel"] & ~amb), nb)
            hi = _rows_to_matrix(orc.expand_pe(r["pe_sel"] | amb), nb)
            excused_total += int(amb.sum())
        got = gpu_matrix(g, h, nb)
        missing = lo & ~got
        extra = got & ~hi
        assert not missing.any(), (h, "missing", np.argwhere(missing)[:8].tolist())
        assert not extra.any(), (h, "extra", np.argwhere(extra)[:8].tolist())
    return excused_total


def check_attention(g, q, k, v, p, samples, key="o", dense=False):
    """Compare sampled query blocks (list of (h, m)) with exact attention over the GPU's lists."""
    hq, hkv = p.n_q_heads, p.n_kv_heads
    B = p.block
    scale = p.softmax_scale if p.softmax_scale > 0 else None
    worst_rel, worst_abs = 0.0, 0.0
    cache = {}
    for h, m in samples:
        kv = orc.kv_head(h, hq, hkv)
        if h not in cache:
            cache = {h: (q[:, h].float().numpy(), k[:, kv].float().numpy(), v[:, kv].float().numpy())}
        qh, kh, vh = cache[h]
        cols = np.arange(m + 1) if dense else gpu_cols(g, h, m)
        want, want_lse = orc.sparse_attention_block(qh, kh, vh, m, cols, B, scale)
        got = g[key][m * B:(m + 1) * B, h]
        err = got - want
        rel = np.linalg.norm(err) / max(np.linalg.norm(want), 1e-30)
        worst_rel = max(worst_rel, rel)
        worst_abs = max(worst_abs, np.abs(err).max())
        assert rel <= 1e-2, (h, m, rel)
        assert np.abs(err).max() <= 2e-2, (h, m, np.abs(err).max())
        lse_key = "lse_dense" if key == "o_dense" else "lse"
        if g.get(lse_key) is not None:
            np.testing.assert_allclose(g[lse_key][h, m * B:(m + 1) * B], want_lse, rtol=1e-3, atol=2e-3)
    return worst_rel, worst_abs


def sample_blocks(nb, hq, per_head, seed=0, always=()):
    """Per head: blocks 0, nb-1 and `always`, plus random ones stratified over four quartiles."""
    rng = np.random.default_rng(seed)
    out = []
    for h in range(hq):
        chosen = {0, nb - 1, *always}
        edges = np.linspace(0, nb, 5).astype(int)
        while len(chosen) < min(per_head, nb):
            for a, b in zip(edges[:-1], edges[1:]):
                if b > a and len(chosen) < per_head:
                    chosen.add(int(rng.integers(a, b)))
        out += [(h, m) for m in sorted(chosen)]
    return out
