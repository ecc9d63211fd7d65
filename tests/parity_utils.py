"""Helpers shared by the GPU parity tests: run the C-ABI stages, run the oracle, compare.

Matching rule (per stage; the list part lives in oracle/matching.py):
  * c_struct, p_v, p_s: floating point, rtol 2e-4 / atol 1e-7 (fp32 accumulation and the hardware
    exp2 approximation against an fp64 oracle).
  * routing labels: identical unless |C_struct - tau| <= 1e-3 * tau.
  * index lists: identical except for blocks whose score lies within 1e-3 (relative) of the deciding
    value (alpha * mu_d, or the value at the k_min / gamma cut).  With A the set of such blocks, the
    GPU list of every query block must lie between expand(S minus A) and expand(S union A).
    For the cumulative rules the entry right at the cut is also excused when the running sum passes
    within 1e-6 of gamma (fp32 scores against fp64).  Both kinds of excused blocks are counted, apart,
    and bounded: at most two mass-band entries per direction and head (the rule cannot produce more),
    and the 1e-3 band may hold at most BAND_LIMIT of a head's candidate blocks.
  * attention output against the oracle's exact attention over the GPU's own lists:
    rel-L2 <= 1e-2 and max-abs <= 2e-2.

The full-size configurations run the oracle in a pool of forked worker processes (one numpy thread each):
most of the oracle's time at 128k tokens and above goes into single-threaded gathers and element-wise
passes, so the host's cores are used by working on several heads / query blocks at once.  The workers
only run numpy on host arrays they inherited; they never touch CUDA.
"""
from __future__ import annotations

import multiprocessing
import os
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

import paper_2609_01925_b200 as crisp
from oracle import crisp_oracle as orc
from oracle import matching

REL_BAND = matching.REL_BAND
MASS_BAND = matching.MASS_BAND
# Largest share of a head's candidate blocks (2 N_b for a VS head, the causal entries for a PE head) that may
# sit inside the 1e-3 band (observed on the Llama-shaped workloads: at most 0.45 %).  Heads with a flat
# background - the sink-dominated heads of Q256k, a diffuse head forced to Vertical-Slash - have all their
# middle blocks within ~1 % of the mean, so several per cent of them lie within 0.1 % of alpha * mu by
# construction of the rule; tests of such inputs pass a wider limit and say why.
BAND_LIMIT = 0.02


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


def _rule_kwargs(p):
    return dict(selector=p.selector, alpha=p.alpha, gamma=p.gamma, k_min=p.k_min_blocks)


class Excused:
    """Blocks excused by the matching rule, counted per head and per kind."""

    def __init__(self):
        self.per_head: Dict[int, Tuple[int, int, int]] = {}   # h -> (band, mass, candidates)

    def add(self, h, band, mass, candidates):
        self.per_head[h] = (int(band), int(mass), int(candidates))

    @property
    def band(self):
        return sum(v[0] for v in self.per_head.values())

    @property
    def mass(self):
        return sum(v[1] for v in self.per_head.values())

    @property
    def worst_band_fraction(self):
        return max((v[0] / max(v[2], 1) for v in self.per_head.values()), default=0.0)

    def __int__(self):
        return self.band + self.mass

    def __str__(self):
        return (f"{self.band} within the 1e-3 band (worst head {100 * self.worst_band_fraction:.2f} % of its "
                f"candidates) + {self.mass} by the 1e-6 mass rule")

    __repr__ = __str__


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


def _check_bounds(h, bounds, band_limit):
    assert max(bounds["mass_per_direction"]) <= 2, (h, "mass rule excused", bounds["mass_per_direction"])
    frac = bounds["band"] / max(bounds["candidates"], 1)
    assert frac <= band_limit, (h, f"{bounds['band']} of {bounds['candidates']} candidate blocks in the 1e-3 band")


def gpu_matrix(g, h, nb):
    """Boolean [N_b, N_b] matrix of the GPU lists of head h; also checks order, bounds and forced blocks."""
    return matching.lists_to_matrix(g["row_ptr"][h], g["col_idx"], nb)


def check_lists(g, res, p, heads=None, band_limit=1.0) -> Excused:
    """GPU lists vs oracle lists under the matching rule.  Returns the excused blocks (int() = their number).
    The share of a head's blocks inside the 1e-3 band is bounded only on request (band_limit): the small and
    degenerate cases that call this directly have a handful of candidate blocks, or ties everywhere."""
    nb = -(-p.seq_len // p.block)
    out = Excused()
    heads = range(len(res)) if heads is None else heads
    for h in heads:
        r = res[h]
        if r is None or g["pattern"][h] != r["pattern"]:
            continue  # label excused by check_route; lists follow the other branch
        bounds = matching.list_bounds(r, nb, **_rule_kwargs(p))
        _check_bounds(h, bounds, band_limit)
        missing, extra = matching.compare_lists(gpu_matrix(g, h, nb), bounds)
        assert not missing, (h, "missing", missing)
        assert not extra, (h, "extra", extra)
        out.add(h, bounds["band"], bounds["mass"], bounds["candidates"])
    return out


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


# ------------------------------------------------------------------------------------------------------
# The same checks with the oracle spread over a pool of forked worker processes (full-size configurations)
# ------------------------------------------------------------------------------------------------------
_CTX: Dict = {}      # set in the parent before the pool forks; read-only in the workers
_CACHE: Dict = {}    # per worker: the fp32 copies of the head it worked on last


def _bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Zero-copy int16 view of a CPU bf16 tensor (numpy has no bf16)."""
    return t.contiguous().view(torch.int16).numpy()


def _head_f32(name: str, h: int) -> np.ndarray:
    bits = _CTX[name][:, h]
    return ((bits.astype(np.uint32) & np.uint32(0xFFFF)) << np.uint32(16)).view(np.float32)


def _worker_head(h: int):
    if _CACHE.get("h") != h:
        kv = orc.kv_head(h, _CTX["hq"], _CTX["hkv"])
        _CACHE.clear()
        _CACHE.update(h=h, q=_head_f32("q", h), k=_head_f32("k", kv), v=_head_f32("v", kv) if "v" in _CTX else None)
    return _CACHE["q"], _CACHE["k"], _CACHE["v"]


def _pool_init():
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:  # pragma: no cover
        pass


def _lists_worker(h: int):
    """Oracle steps O1-O6 of one head and the comparison of its lists; returns only small results."""
    qh, kh, _ = _worker_head(h)
    kw, rule, nb = _CTX["oracle_kw"], _CTX["rule_kw"], _CTX["nb"]
    r = orc.head_pipeline(qh, kh, **kw)
    out = dict(h=h, c_struct=r["c_struct"], pattern=r["pattern"], p_v=r["p_v"], p_s=r["p_s"])
    for key in ("s_v", "s_s", "k_v", "k_s", "raw_v", "raw_s", "pe_cut"):
        if key in r:
            out[key] = r[key]
    if _CTX["pattern"][h] != r["pattern"]:
        out["skipped"] = True      # the label differs: check_route decides whether that is excused
        return out
    bounds = matching.list_bounds(r, nb, **rule)
    got = matching.lists_to_matrix(_CTX["row_ptr"][h], _CTX["col_idx"], nb)
    missing, extra = matching.compare_lists(got, bounds)
    out.update(band=bounds["band"], mass=bounds["mass"], candidates=bounds["candidates"],
               mass_per_direction=bounds["mass_per_direction"], missing=missing, extra=extra)
    return out


def _attention_worker(task):
    h, m, cols, got, got_lse = task
    qh, kh, vh = _worker_head(h)
    want, want_lse = orc.sparse_attention_block(qh, kh, vh, m, cols, _CTX["block"], _CTX["scale"])
    err = got - want
    rel = float(np.linalg.norm(err) / max(np.linalg.norm(want), 1e-30))
    lse_err = None
    if got_lse is not None:
        lse_err = float(np.max(np.abs(got_lse - want_lse) - 1e-3 * np.abs(want_lse)))
    return h, m, rel, float(np.abs(err).max()), lse_err


class OraclePool:
    """Worker processes that share the host copies of Q, K, V (and the GPU's lists) by fork."""

    def __init__(self, p, qc, kc, vc=None, g=None, workers: Optional[int] = None):
        _CTX.clear()
        _CTX.update(q=_bf16_bits(qc), k=_bf16_bits(kc), hq=p.n_q_heads, hkv=p.n_kv_heads, block=p.block,
                    nb=-(-p.seq_len // p.block), scale=(p.softmax_scale if p.softmax_scale > 0 else None),
                    oracle_kw=oracle_kwargs(p), rule_kw=_rule_kwargs(p))
        if vc is not None:
            _CTX["v"] = _bf16_bits(vc)
        if g is not None:
            _CTX.update(pattern=g["pattern"], row_ptr=g["row_ptr"], col_idx=g["col_idx"])
        n = workers or min(os.cpu_count() or 1, 16)
        self.pool = multiprocessing.get_context("fork").Pool(n, initializer=_pool_init)
        self.p = p

    def close(self):
        self.pool.close()
        self.pool.join()
        _CTX.clear()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def heads(self, g, heads: Sequence[int], band_limit=BAND_LIMIT):
        """Routing and lists of `heads` against the oracle.  Returns (per-head oracle results (small parts
        only), excused labels, Excused)."""
        p = self.p
        # heads routed to pooled estimation cost ten times more: start them first
        order = sorted(heads, key=lambda h: (g["pattern"][h] != orc.PE, h))
        res: List[Optional[Dict]] = [None] * p.n_q_heads
        for out in self.pool.imap_unordered(_lists_worker, order):
            res[out["h"]] = out
        labels = check_route(g, res, p, heads=heads)
        exc = Excused()
        for h in heads:
            r = res[h]
            if r.get("skipped"):
                continue
            _check_bounds(h, r, band_limit)
            assert not r["missing"], (h, "missing", r["missing"])
            assert not r["extra"], (h, "extra", r["extra"])
            exc.add(h, r["band"], r["mass"], r["candidates"])
        return res, labels, exc

    def attention(self, g, samples, fetch_block, lse=None, dense=False):
        """Sampled query blocks (h, m) against exact attention over the GPU's lists (or every causal block).
        fetch_block(h, m) returns the GPU output of the block as float32 [rows, 128]."""
        B = self.p.block
        tasks = []
        for h, m in samples:
            cols = np.arange(m + 1) if dense else np.asarray(gpu_cols(g, h, m))
            got = fetch_block(h, m)
            got_lse = None if lse is None else np.asarray(lse[h, m * B:m * B + got.shape[0]])
            tasks.append((h, m, cols, got, got_lse))
        # longest lists first, grouped by head so that a worker converts a head's Q, K, V once per chunk
        per_head = {}
        for t in tasks:
            per_head[t[0]] = per_head.get(t[0], 0) + len(t[2])
        tasks.sort(key=lambda t: (-per_head[t[0]], t[0], -len(t[2])))
        worst_rel = worst_abs = 0.0
        blocks = 0
        for h, m, rel, mab, lse_err in self.pool.imap_unordered(_attention_worker, tasks, chunksize=2):
            assert rel <= 1e-2, (h, m, rel)
            assert mab <= 2e-2, (h, m, mab)
            assert lse_err is None or lse_err <= 2e-3, (h, m, "lse", lse_err)
            worst_rel, worst_abs = max(worst_rel, rel), max(worst_abs, mab)
        for t in tasks:
            blocks += len(t[2])
        return worst_rel, worst_abs, blocks
