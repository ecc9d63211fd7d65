"""The GPU <-> oracle matching rule for routing labels and index lists (numpy).

TEST INFRASTRUCTURE ONLY, like the rest of this folder: the tests and the benchmark's CPU-baseline leg use
it to decide which differences between the CUDA path's lists and the oracle's are excused, and to count them.
It holds no arithmetic of the method beyond calls into crisp_oracle.

Rule.  A block's membership may differ only when its score lies within REL_BAND (relative) of the value that
decides it: alpha * mu_d for the noise-floor rules, the values on either side of the k_min or gamma cut for
the ranked rules, the value at the cut of the pooled map.  For the cumulative rules (Algorithm 6, Algorithm 4)
one more entry is excused when the running mass passes within MASS_BAND of gamma: the CUDA path sums fp32
scores, the oracle fp64 ones, and a difference of ~1e-7 in the running sum can move the cut by one entry.
With A the set of excused blocks, every list of the CUDA path must lie between expand(S minus A) and
expand(S union A).  The two kinds of excuse are counted apart.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np

from . import crisp_oracle as orc

REL_BAND = 1e-3
MASS_BAND = 1e-6


def ambiguous_vs(pd: np.ndarray, k_d: int, raw: int, *, selector: int, alpha: float, gamma: float,
                 k_min: int) -> Tuple[np.ndarray, np.ndarray]:
    """Blocks of one direction whose membership may differ: (within REL_BAND of the deciding value,
    excused by the MASS_BAND rule)."""
    nb = pd.shape[0]
    order = np.argsort(-pd, kind="stable")
    band = np.zeros(nb, dtype=bool)
    mass = np.zeros(nb, dtype=bool)
    if selector in (0, 2):
        mu = orc.noise_floor(pd)[1] if selector == 0 else float(np.median(pd[1:nb - 1]))
        thr = alpha * mu
        band |= np.abs(pd - thr) <= REL_BAND * thr
    if selector == 1 and raw < nb:
        cs = np.cumsum(pd[order])
        if cs[raw - 1] - gamma <= MASS_BAND:
            mass[order[raw]] = True
        if raw >= 2 and gamma - cs[raw - 2] <= MASS_BAND:
            mass[order[raw - 1]] = True
    if selector == 1 or raw < k_min:
        if k_d < nb:
            cut = pd[order[k_d - 1]]
            band |= np.abs(pd - cut) <= REL_BAND * cut
            nxt = pd[order[k_d]]
            band |= np.abs(pd - nxt) <= REL_BAND * max(nxt, 1e-300)
    mass &= ~band
    return band, mass


def _rows_to_matrix(cols_per_row, nb: int) -> np.ndarray:
    m = np.zeros((nb, nb), dtype=bool)
    for r, c in enumerate(cols_per_row):
        m[r, c] = True
    return m


def list_bounds(res: Dict, nb: int, *, selector: int, alpha: float, gamma: float, k_min: int) -> Dict:
    """Lower and upper bound (boolean [N_b, N_b]) of the lists of one head, from the oracle's result `res`
    (crisp_oracle.head_pipeline), and the number of excused and candidate blocks."""
    if nb <= 2:
        lo = hi = _rows_to_matrix(res["cols"], nb)
        return dict(lo=lo, hi=hi, band=0, mass=0, candidates=nb, mass_per_direction=(0, 0))
    if res["pattern"] == orc.VS:
        kw = dict(selector=selector, alpha=alpha, gamma=gamma, k_min=k_min)
        band_v, mass_v = ambiguous_vs(res["p_v"], res["k_v"], res["raw_v"], **kw)
        band_s, mass_s = ambiguous_vs(res["p_s"], res["k_s"], res["raw_s"], **kw)
        amb_v, amb_s = band_v | mass_v, band_s | mass_s
        sv = np.zeros(nb, bool); sv[res["s_v"]] = True
        ss = np.zeros(nb, bool); ss[res["s_s"]] = True
        lo = _rows_to_matrix(orc.expand_vs(np.nonzero(sv & ~amb_v)[0], np.nonzero(ss & ~amb_s)[0], nb), nb)
        hi = _rows_to_matrix(orc.expand_vs(np.nonzero(sv | amb_v)[0], np.nonzero(ss | amb_s)[0], nb), nb)
        return dict(lo=lo, hi=hi, band=int(band_v.sum() + band_s.sum()), mass=int(mass_v.sum() + mass_s.sum()),
                    candidates=2 * nb, mass_per_direction=(int(mass_v.sum()), int(mass_s.sum())))
    flat = res["a_bar"] / res["a_bar"].sum()
    cut = res["pe_cut"]
    tri = np.tril(np.ones((nb, nb), bool))
    band = (np.abs(flat - cut) <= REL_BAND * cut) & tri
    mass = np.zeros((nb, nb), bool)
    vals = np.where(tri, flat, -1.0).reshape(-1)
    order = np.argsort(-vals, kind="stable")[:int(tri.sum())]
    cs = np.cumsum(vals[order])
    kstar = int(res["pe_sel"].sum())
    if kstar < order.size and cs[kstar - 1] - gamma <= MASS_BAND:
        mass.reshape(-1)[order[kstar]] = True
    if kstar >= 2 and gamma - cs[kstar - 2] <= MASS_BAND:
        mass.reshape(-1)[order[kstar - 1]] = True
    mass &= ~band
    amb = band | mass
    lo = _rows_to_matrix(orc.expand_pe(res["pe_sel"] & ~amb), nb)
    hi = _rows_to_matrix(orc.expand_pe(res["pe_sel"] | amb), nb)
    return dict(lo=lo, hi=hi, band=int(band.sum()), mass=int(mass.sum()), candidates=int(tri.sum()),
                mass_per_direction=(int(mass.sum()), 0))


def lists_to_matrix(row_ptr_h: np.ndarray, col_idx: np.ndarray, nb: int) -> np.ndarray:
    """Boolean [N_b, N_b] matrix of one head's CSR lists (row_ptr_h holds global offsets into col_idx); checks
    that every row is ascending, unique, within [0, m] and holds its forced blocks 0 and m."""
    rp = np.asarray(row_ptr_h, dtype=np.int64)
    cols = np.asarray(col_idx[rp[0]:rp[nb]], dtype=np.int64)
    lens = np.diff(rp)
    rows = np.repeat(np.arange(nb), lens)
    assert lens.min() >= 1, "empty row"
    assert np.all(cols <= rows) and np.all(cols >= 0), "column out of range"
    same_row = rows[1:] == rows[:-1]
    assert np.all(np.diff(cols)[same_row] > 0), "not ascending/unique"
    first = rp[:-1] - rp[0]
    last = rp[1:] - rp[0] - 1
    assert np.all(cols[first] == 0) and np.all(cols[last] == np.arange(nb)), "forced blocks missing"
    m = np.zeros((nb, nb), dtype=bool)
    m[rows, cols] = True
    return m


def compare_lists(got: np.ndarray, bounds: Dict) -> Tuple[List, List]:
    """(missing, extra): entries of the lower bound the lists lack, entries beyond the upper bound."""
    missing = bounds["lo"] & ~got
    extra = got & ~bounds["hi"]
    return np.argwhere(missing)[:8].tolist(), np.argwhere(extra)[:8].tolist()
