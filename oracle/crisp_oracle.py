"""Plain fp64 CPU oracle of CRISP's sparse-prefill path (numpy).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this file;
only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
It shares no code with the CUDA library: it is written from the paper's
definitions, step by step, with numpy matmul / sort / cumsum as library steps
and no blocking, fusion or reordering beyond what the definitions state.

Sequence lengths need not be multiples of the block size: N_b = ceil(n / B) as in Section 4.3, the last
block simply holds fewer tokens.

Conventions (one attention layer):
  q [n, H_q, d], k, v [n, H_kv, d]: arrays holding bf16-representable values
  (float32 or float64); query head h reads KV head h // (H_q // H_kv).
  B = block size, N_b = n / B, the proxy queries are the last B tokens, proxy
  row i is token t_i = n - B + i.

Pins (tests/test_oracle_*.py): closed forms for uniform / one-hot / two-level
logits (Appendix C), brute-force loops on tiny inputs, fp64 library attention,
hand-computed toy vectors for the noise floor and both gamma failure modes,
invariants (unit mass, alpha monotonicity, always-kept blocks, token-level
cover).  The paper prints no worked numerical example of Algorithms 2-4, so the
end-to-end pipeline has no printed value to match: parity of the pipeline as a
whole against the paper's own numbers is unpinned; every step is pinned
separately as listed.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np

VS, PE = 1, 0


def _head(x: np.ndarray, h: int) -> np.ndarray:
    return np.asarray(x[:, h, :], dtype=np.float64)


def kv_head(h: int, n_q_heads: int, n_kv_heads: int) -> int:
    return h // (n_q_heads // n_kv_heads)


# ----------------------------------------------------------------------------------------
# Algorithm 2, lines 3-5: representative queries and proxy attention
# ----------------------------------------------------------------------------------------
def proxy_attention(q_h: np.ndarray, k_h: np.ndarray, block: int,
                    scale: float | None = None) -> np.ndarray:
    """A_hat = Softmax(Q_hat K^T / sqrt(d)) for Q_hat = the last `block` queries.

    q_h [n, d], k_h [n, d] (one query head and its KV head).  The map is causal:
    row i (token t_i) sees keys j <= t_i; masked entries are exactly 0.
    Returns [block, n] fp64, rows summing to 1.
    """
    q_h = np.asarray(q_h, dtype=np.float64)
    k_h = np.asarray(k_h, dtype=np.float64)
    n, d = k_h.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    q_hat = q_h[n - block:]
    s = (q_hat @ k_h.T) * scale
    t = (n - block) + np.arange(block)[:, None]
    j = np.arange(n)[None, :]
    s = np.where(j <= t, s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------------------------------
# Eq. 2 / Algorithm 2, lines 6-12: structural mass and the routing gate
# ----------------------------------------------------------------------------------------
def c_struct(a_hat: np.ndarray, sink_tokens: int, local_tokens: int) -> float:
    """Mean over proxy rows of the mass on the anchor positions.

    Anchors: the first `sink_tokens` keys and the last `local_tokens` keys of the
    sequence (absolute positions); a key in both windows counts once.
    """
    b, n = a_hat.shape
    anchor = np.zeros(n, dtype=bool)
    anchor[:min(sink_tokens, n)] = True
    anchor[max(n - local_tokens, 0):] = True
    return float(a_hat[:, anchor].sum() / b)


def route(c: float, tau: float) -> int:
    """VS iff C_struct >= tau_proxy (Algorithm 2)."""
    return VS if c >= tau else PE


# ----------------------------------------------------------------------------------------
# Algorithm 5 (Appendix A): the Jensen-Shannon router that C_struct replaces (comparison only)
# ----------------------------------------------------------------------------------------
def js_distance(a: np.ndarray, b: np.ndarray) -> float:
    """sqrt(0.5 KL(a || m) + 0.5 KL(b || m)), m = (a + b) / 2; natural log, 0 log 0 = 0."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    m = 0.5 * (a + b)
    kl_a = np.sum(np.where(a > 0, a * np.log(np.where(a > 0, a, 1.0) / np.where(m > 0, m, 1.0)), 0.0))
    kl_b = np.sum(np.where(b > 0, b * np.log(np.where(b > 0, b, 1.0) / np.where(m > 0, m, 1.0)), 0.0))
    return float(math.sqrt(max(0.5 * kl_a + 0.5 * kl_b, 0.0)))


def jsd_router(q_h: np.ndarray, k_h: np.ndarray, block: int, scale: float | None = None) -> Tuple[float, np.ndarray, np.ndarray]:
    """(D_JS, a_bar, a_hat): a_bar = Softmax(pool(Q_hat) pool(K)^T / sqrt(d)) over the key blocks
    (pool = mean over the block's rows), a_hat = block sums of the mean proxy row (= p_v)."""
    q_h = np.asarray(q_h, dtype=np.float64)
    k_h = np.asarray(k_h, dtype=np.float64)
    n, d = k_h.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    q_bar = q_h[n - block:].mean(axis=0)
    k_bar = block_means(k_h, block)
    z = (k_bar @ q_bar) * scale
    e = np.exp(z - z.max())
    a_bar = e / e.sum()
    a_hat, _ = block_scores(proxy_attention(q_h, k_h, block, scale), block)
    return js_distance(a_hat, a_bar), a_bar, a_hat


# ----------------------------------------------------------------------------------------
# Algorithm 3, lines 3-5 (normalisation as in Algorithm 6, lines 2-3): block scores
# ----------------------------------------------------------------------------------------
def block_scores(a_hat: np.ndarray, block: int) -> Tuple[np.ndarray, np.ndarray]:
    """p_v, p_s: block-pooled vertical (column) and slash (diagonal) mass, each summing to 1.

    a_v[j] = sum_i A[i, j] / sum(A); a_s[o] = sum over entries with t_i - j = o, / sum(A);
    pooling adds the `block` consecutive entries of a block.  sum(A) = number of rows.
    """
    b, n = a_hat.shape
    nb = -(-n // block)                      # N_b = ceil(n / B); the last block may be partial
    total = a_hat.sum()
    a_v = a_hat.sum(axis=0) / total
    a_s = np.zeros(n, dtype=np.float64)
    for i in range(b):
        t = n - b + i
        # offset o = t - j for j = 0..t  <=>  reversed visible part of the row
        a_s[:t + 1] += a_hat[i, t::-1]
    a_s /= total
    starts = np.arange(0, n, block)
    p_v = np.add.reduceat(a_v, starts)
    p_s = np.add.reduceat(a_s, starts)
    assert p_v.shape[0] == nb
    return p_v, p_s


# ----------------------------------------------------------------------------------------
# Algorithm 3, lines 6-12 / Eq. 3-4: sink-aware noise-floor budget
# ----------------------------------------------------------------------------------------
def noise_floor(p: np.ndarray) -> Tuple[float, float]:
    """(r, mu): residual mass outside the first and last block, and its mean per block.

    r = max(1 - p[0] - p[N_b-1], 0), evaluated as the sum of the middle blocks (the two
    agree exactly for a unit-mass p; the sum has no cancellation when sinks hold ~1).
    """
    nb = p.shape[0]
    r = float(p[1:nb - 1].sum())
    return r, r / (nb - 2)


def stable_topk(p: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries, ties broken towards the lower index."""
    order = np.argsort(-p, kind="stable")
    return order[:k]


def select_noise_floor(p: np.ndarray, alpha: float, k_min: int) -> Tuple[np.ndarray, int, int]:
    """Top-k_d blocks with k_d = clip(#{p > alpha * mu}, k_min, N_b).

    Returns (sorted block indices, k_d after clipping, raw count before clipping).
    """
    nb = p.shape[0]
    _, mu = noise_floor(p)
    raw = int(np.count_nonzero(p > alpha * mu))
    k_d = min(max(raw, k_min), nb)
    return np.sort(stable_topk(p, k_d)), k_d, raw


def select_median_floor(p: np.ndarray, alpha: float, k_min: int) -> Tuple[np.ndarray, int, int]:
    """Appendix H variant: the floor is the MEDIAN mass of the non-retained blocks instead of their mean.

    k_d = clip(#{p > alpha * median(p[1 : N_b-1])}, k_min, N_b); the rest is Algorithm 3 unchanged.
    """
    nb = p.shape[0]
    med = float(np.median(p[1:nb - 1]))
    raw = int(np.count_nonzero(p > alpha * med))
    k_d = min(max(raw, k_min), nb)
    return np.sort(stable_topk(p, k_d)), k_d, raw


# ----------------------------------------------------------------------------------------
# Algorithm 6, lines 4-5: cumulative-gamma budget (comparison selector)
# ----------------------------------------------------------------------------------------
def gamma_count(sorted_desc: np.ndarray, gamma: float) -> int:
    """Smallest k with sum of the k largest >= gamma; all entries if never reached."""
    cs = np.cumsum(sorted_desc)
    hit = np.nonzero(cs >= gamma)[0]
    return int(hit[0]) + 1 if hit.size else int(sorted_desc.shape[0])


def select_gamma(p: np.ndarray, gamma: float, k_min: int) -> Tuple[np.ndarray, int, int]:
    """Top-k_d blocks with k_d = clip(min{k: cumsum_k >= gamma}, k_min, N_b)."""
    nb = p.shape[0]
    order = np.argsort(-p, kind="stable")
    raw = gamma_count(p[order], gamma)
    k_d = min(max(raw, k_min), nb)
    return np.sort(order[:k_d]), k_d, raw


# ----------------------------------------------------------------------------------------
# Algorithm 4: pooled estimation (PE) index set
# ----------------------------------------------------------------------------------------
def block_means(x: np.ndarray, block: int) -> np.ndarray:
    """Mean over the rows of every block of `block` tokens (the last block may hold fewer rows)."""
    n = x.shape[0]
    starts = np.arange(0, n, block)
    counts = np.minimum(starts + block, n) - starts
    return np.add.reduceat(x, starts, axis=0) / counts[:, None]


def pooled_map(q_h: np.ndarray, k_h: np.ndarray, block: int,
               scale: float | None = None) -> np.ndarray:
    """A_bar = row softmax of pool(Q) pool(K)^T / sqrt(d), causal at block level (J <= m).

    pool = mean over the block's rows.  Returns [N_b, N_b] fp64, non-causal entries 0.
    """
    q_h = np.asarray(q_h, dtype=np.float64)
    k_h = np.asarray(k_h, dtype=np.float64)
    n, d = q_h.shape
    nb = -(-n // block)
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    q_bar = block_means(q_h, block)
    k_bar = block_means(k_h, block)
    z = (q_bar @ k_bar.T) * scale
    m = np.arange(nb)[:, None]
    jj = np.arange(nb)[None, :]
    z = np.where(jj <= m, z, -np.inf)
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=1, keepdims=True)


def select_pe(a_bar: np.ndarray, gamma: float) -> Tuple[np.ndarray, float]:
    """Flatten, normalise by the total, sort descending (stable), keep the shortest prefix
    whose mass reaches gamma.  Returns (boolean [N_b, N_b] selection, value at the cut)."""
    nb = a_bar.shape[0]
    flat = (a_bar / a_bar.sum()).reshape(-1)
    causal = (np.arange(nb)[None, :] <= np.arange(nb)[:, None]).reshape(-1)
    order = np.argsort(-flat, kind="stable")
    order = order[causal[order]]                      # non-causal entries do not exist
    k_star = gamma_count(flat[order], gamma)
    sel = np.zeros(nb * nb, dtype=bool)
    sel[order[:k_star]] = True
    return sel.reshape(nb, nb), float(flat[order[k_star - 1]])


# ----------------------------------------------------------------------------------------
# Expansion of the per-head sets into per-query-block key-block lists (Eq. 1's S_i)
# ----------------------------------------------------------------------------------------
def expand_vs(s_v: Sequence[int], s_s: Sequence[int], nb: int) -> List[np.ndarray]:
    """cols(m) = {0, m} u {J in S_v, J <= m} u ({m-s, m-s-1 : s in S_s} n [0, m]).

    Vertical indices are absolute key blocks; slash indices are block offsets: the token
    band of offsets [sB, sB+B) of query block m touches key blocks m-s and m-s-1.
    """
    s_v = np.asarray(s_v, dtype=np.int64)
    s_s = np.asarray(s_s, dtype=np.int64)
    out = []
    for m in range(nb):
        keep = np.zeros(m + 1, dtype=bool)
        keep[0] = True
        keep[m] = True
        keep[s_v[s_v <= m]] = True
        a = m - s_s
        keep[a[(a >= 0)]] = True
        a = a - 1
        keep[a[(a >= 0)]] = True
        out.append(np.nonzero(keep)[0].astype(np.int32))
    return out


def expand_pe(sel: np.ndarray) -> List[np.ndarray]:
    """cols(m) = {0, m} u {J <= m : (m, J) selected}."""
    nb = sel.shape[0]
    out = []
    for m in range(nb):
        keep = sel[m, :m + 1].copy()
        keep[0] = True
        keep[m] = True
        out.append(np.nonzero(keep)[0].astype(np.int32))
    return out


def dense_cols(nb: int) -> List[np.ndarray]:
    return [np.arange(m + 1, dtype=np.int32) for m in range(nb)]


# ----------------------------------------------------------------------------------------
# Eq. 1: exact softmax attention restricted to the selected blocks, causal
# ----------------------------------------------------------------------------------------
def sparse_attention_block(q_h: np.ndarray, k_h: np.ndarray, v_h: np.ndarray, m: int,
                           cols: Sequence[int], block: int,
                           scale: float | None = None) -> Tuple[np.ndarray, np.ndarray]:
    """Output rows of query block m attending to the key blocks in `cols`, keys j <= t.

    Returns (O [block, d] fp64, lse [block] fp64 = log sum exp of the kept scaled logits).
    """
    n = np.asarray(k_h).shape[0]
    q_h = np.asarray(q_h[m * block:min((m + 1) * block, n)], dtype=np.float64)
    d = q_h.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    cols = np.asarray(cols, dtype=np.int64)
    key_idx = (cols[:, None] * block + np.arange(block)[None, :]).reshape(-1)
    key_idx = key_idx[key_idx < n]           # the last key block may be partial
    kk = np.asarray(k_h[key_idx], dtype=np.float64)
    vv = np.asarray(v_h[key_idx], dtype=np.float64)
    s = (q_h @ kk.T) * scale
    t = m * block + np.arange(q_h.shape[0])[:, None]
    s = np.where(key_idx[None, :] <= t, s, -np.inf)
    mx = s.max(axis=1, keepdims=True)
    e = np.exp(s - mx)
    l = e.sum(axis=1, keepdims=True)
    o = (e / l) @ vv
    return o, (mx + np.log(l)).reshape(-1)


def sparse_attention_head(q_h, k_h, v_h, cols_per_block: Sequence[Sequence[int]], block: int,
                          scale: float | None = None) -> Tuple[np.ndarray, np.ndarray]:
    n, d = np.asarray(q_h).shape
    o = np.empty((n, d), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    for m, cols in enumerate(cols_per_block):
        hi = min((m + 1) * block, n)
        o[m * block:hi], lse[m * block:hi] = sparse_attention_block(q_h, k_h, v_h, m, cols, block, scale)
    return o, lse


# ----------------------------------------------------------------------------------------
# Algorithm 1: the whole per-head pipeline up to the index lists
# ----------------------------------------------------------------------------------------
def head_pipeline(q_h: np.ndarray, k_h: np.ndarray, *, block: int = 128, sink_tokens: int = 128,
                  local_tokens: int = 128, tau: float = 0.2, alpha: float = 1.0,
                  gamma: float = 0.95, k_min_blocks: int = 8, selector: int = 0,
                  force_pattern: int = 0, scale: float | None = None) -> Dict:
    """Route one head and build its per-query-block key-block lists.

    selector 0 = noise floor (Algorithm 3), 1 = cumulative gamma (Algorithm 6), 2 = median floor
    (Appendix H); VS heads only.
    force_pattern 0 = by C_struct, 1 = VS, 2 = PE.
    """
    n = np.asarray(q_h).shape[0]
    nb = -(-n // block)
    a_hat = proxy_attention(q_h, k_h, block, scale)
    c = c_struct(a_hat, sink_tokens, local_tokens)
    pattern = route(c, tau)
    if force_pattern == 1:
        pattern = VS
    elif force_pattern == 2:
        pattern = PE
    p_v, p_s = block_scores(a_hat, block)
    res = dict(c_struct=c, pattern=pattern, p_v=p_v, p_s=p_s)
    if nb <= 2:
        res["cols"] = dense_cols(nb)
        return res
    if pattern == VS:
        if selector == 0:
            s_v, kv_, raw_v = select_noise_floor(p_v, alpha, k_min_blocks)
            s_s, ks_, raw_s = select_noise_floor(p_s, alpha, k_min_blocks)
        elif selector == 2:
            s_v, kv_, raw_v = select_median_floor(p_v, alpha, k_min_blocks)
            s_s, ks_, raw_s = select_median_floor(p_s, alpha, k_min_blocks)
        else:
            s_v, kv_, raw_v = select_gamma(p_v, gamma, k_min_blocks)
            s_s, ks_, raw_s = select_gamma(p_s, gamma, k_min_blocks)
        res.update(s_v=s_v, s_s=s_s, k_v=kv_, k_s=ks_, raw_v=raw_v, raw_s=raw_s)
        res["cols"] = expand_vs(s_v, s_s, nb)
    else:
        a_bar = pooled_map(q_h, k_h, block, scale)
        sel, cut = select_pe(a_bar, gamma)
        res.update(a_bar=a_bar, pe_sel=sel, pe_cut=cut)
        res["cols"] = expand_pe(sel)
    return res


def layer_pipeline(q, k, **kw) -> List[Dict]:
    """head_pipeline for every query head of a layer (GQA: head h reads KV head h // G)."""
    n, hq, _ = q.shape
    hkv = k.shape[1]
    return [head_pipeline(_head(q, h), _head(k, kv_head(h, hq, hkv)), **kw) for h in range(hq)]


def cols_to_csr(cols_per_head: Sequence[Sequence[np.ndarray]]) -> Tuple[np.ndarray, np.ndarray]:
    """Flat CSR over (head, query block): row_ptr [H, N_b+1] (global offsets), col_idx."""
    hq = len(cols_per_head)
    nb = len(cols_per_head[0])
    row_ptr = np.zeros((hq, nb + 1), dtype=np.int64)
    chunks = []
    off = 0
    for h in range(hq):
        for m in range(nb):
            row_ptr[h, m] = off
            chunks.append(np.asarray(cols_per_head[h][m], dtype=np.int32))
            off += chunks[-1].shape[0]
        row_ptr[h, nb] = off
    return row_ptr, (np.concatenate(chunks) if chunks else np.zeros(0, np.int32))
