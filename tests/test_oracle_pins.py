"""Pins of the fp64 oracle against closed forms, brute force and library routines.

Each test names the passage of the paper whose definition it checks.  None of them
retypes the oracle's own formula: they use closed forms, independent loops, hand-worked
fixtures (tests/golden) or torch's fp64 attention.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import crisp_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
B = 16  # small block for most pins (the oracle is generic in the block size)


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ O1 proxy (Algorithm 2)
def test_proxy_uniform_when_keys_zero():
    n, d = 8 * B, 8
    q = rng(0).normal(size=(n, d))
    a = orc.proxy_attention(q, np.zeros((n, d)), B)
    for i in range(B):
        t = n - B + i
        assert np.allclose(a[i, :t + 1], 1.0 / (t + 1), rtol=1e-14)
        assert np.all(a[i, t + 1:] == 0.0)


def test_proxy_two_level_logits_appendix_c():
    """k signal keys at logit z, the rest at z - Delta: background mass eps (Appendix C)."""
    vals = {}
    with open(os.path.join(GOLDEN, "gamma_failure_modes.txt")) as f:
        for line in f:
            if line.startswith("two_level"):
                tok = line.split()
                vals = {tok[i]: float(tok[i + 1]) for i in range(1, len(tok), 2)}
    k_sig, n, delta, eps_gold = int(vals["k"]), int(vals["n"]), vals["delta"], vals["eps"]
    d = 16
    blk = 128
    scale = 1.0 / math.sqrt(d)
    q = np.zeros((n, d)); q[:, 0] = 4.0            # c = 4, exactly representable
    k = np.zeros((n, d)); k[:, 0] = 0.0            # background: logit 0
    sig = [0, 1, 2, 3]
    k[sig, 0] = delta / (4.0 * scale)              # signal: logit = 4 * x * scale = delta
    a = orc.proxy_attention(q, k, blk)
    last = a[blk - 1]                               # sees all n keys
    assert np.isclose(last[100], eps_gold, rtol=1e-8)
    for i in (0, 17, blk - 1):
        ni = n - blk + i + 1
        eps = math.exp(-delta) / (k_sig + (ni - k_sig) * math.exp(-delta))
        assert np.isclose(a[i, 500], eps, rtol=1e-12)
        assert np.isclose(a[i, 0], eps * math.exp(delta), rtol=1e-12)


def test_proxy_bruteforce_loops():
    n, d, blk = 64, 4, 8
    r = rng(1)
    q, k = r.normal(size=(n, d)), r.normal(size=(n, d))
    a = orc.proxy_attention(q, k, blk)
    for i in range(blk):
        t = n - blk + i
        logits = [sum(q[t, c] * k[j, c] for c in range(d)) / math.sqrt(d) for j in range(t + 1)]
        mx = max(logits)
        den = sum(math.exp(x - mx) for x in logits)
        for j in range(n):
            want = math.exp(logits[j] - mx) / den if j <= t else 0.0
            assert abs(a[i, j] - want) < 1e-14


def test_proxy_custom_scale():
    n, d, blk = 32, 4, 8
    r = rng(2)
    q, k = r.normal(size=(n, d)), r.normal(size=(n, d))
    a1 = orc.proxy_attention(q, k, blk, scale=0.25)
    a2 = orc.proxy_attention(q * 0.5, k, blk, scale=0.5)
    assert np.allclose(a1, a2, rtol=1e-13, atol=0)


# ------------------------------------------------------------------ O2 C_struct (Eq. 2)
def uniform_map(n, blk):
    a = np.zeros((blk, n))
    for i in range(blk):
        t = n - blk + i
        a[i, :t + 1] = 1.0 / (t + 1)
    return a


@pytest.mark.parametrize("w_sink", [1, 4, 16])
def test_c_struct_uniform_closed_form(w_sink):
    n = 12 * B
    a = uniform_map(n, B)
    want = sum((min(w_sink, n - B + i + 1) + (i + 1)) / (n - B + i + 1) for i in range(B)) / B
    assert np.isclose(orc.c_struct(a, w_sink, B), want, rtol=1e-13)


def test_c_struct_one_hot_membership():
    n = 10 * B
    for j_star, want in [(0, 1.0), (3, 1.0), (4, 0.0), (5 * B, 0.0), (n - B - 1, 0.0), (n - B, 1.0)]:
        a = np.zeros((B, n)); a[:, j_star] = 1.0
        assert orc.c_struct(a, 4, B) == want
    # a key inside both windows is counted once
    a = np.zeros((B, 2 * B)); a[:, B + 1] = 1.0
    assert orc.c_struct(a, 2 * B, B) == 1.0


def test_c_struct_equals_first_plus_last_block_when_windows_are_blocks():
    """Section 4.3: with w_sink = w_local = B the anchors are exactly the first and last block."""
    n, d = 9 * B, 8
    r = rng(3)
    a = orc.proxy_attention(r.normal(size=(n, d)) * 2, r.normal(size=(n, d)) * 2, B)
    p_v, _ = orc.block_scores(a, B)
    assert np.isclose(orc.c_struct(a, B, B), p_v[0] + p_v[-1], rtol=1e-13)


def test_route_gate_is_geq():
    assert orc.route(0.2, 0.2) == orc.VS
    assert orc.route(0.19999, 0.2) == orc.PE


# ------------------------------------------------------------------ O3 block scores (Alg. 3 l.3-5)
def test_block_scores_unit_mass():
    n, d = 7 * B, 8
    r = rng(4)
    a = orc.proxy_attention(r.normal(size=(n, d)), r.normal(size=(n, d)), B)
    p_v, p_s = orc.block_scores(a, B)
    assert np.isclose(p_v.sum(), 1.0, rtol=1e-13) and np.isclose(p_s.sum(), 1.0, rtol=1e-13)
    assert p_v.shape == p_s.shape == (7,)


@pytest.mark.parametrize("J,c", [(0, 0), (2, 5), (4, B - 1), (6, 0)])
def test_block_scores_one_hot_column(J, c):
    nb = 8
    n = nb * B
    a = np.zeros((B, n)); a[:, J * B + c] = 1.0
    p_v, p_s = orc.block_scores(a, B)
    e = np.zeros(nb); e[J] = 1.0
    assert np.array_equal(p_v, e)
    assert np.isclose(p_s[nb - 1 - J], (B - c) / B)
    if c:
        assert np.isclose(p_s[nb - 2 - J], c / B)
    assert np.isclose(p_s.sum(), 1.0)


@pytest.mark.parametrize("delta", [0, 1, B - 1, B, 3 * B + 5])
def test_block_scores_planted_diagonal(delta):
    nb = 8
    n = nb * B
    a = np.zeros((B, n))
    for i in range(B):
        a[i, n - B + i - delta] = 1.0
    p_v, p_s = orc.block_scores(a, B)
    e = np.zeros(nb); e[delta // B] = 1.0
    assert np.allclose(p_s, e)
    rem = delta % B
    # keys n-B-delta .. n-1-delta: `rem` of them fall in the lower key block
    top = (n - 1 - delta) // B
    assert np.isclose(p_v[top], (B - rem) / B)
    if rem:
        assert np.isclose(p_v[top - 1], rem / B)


def test_block_scores_bruteforce_loops():
    n, d, blk = 48, 4, 8
    r = rng(5)
    a = orc.proxy_attention(r.normal(size=(n, d)), r.normal(size=(n, d)), blk)
    nb = n // blk
    pv = [0.0] * nb
    ps = [0.0] * nb
    for i in range(blk):
        t = n - blk + i
        for j in range(t + 1):
            pv[j // blk] += a[i, j] / blk
            ps[(t - j) // blk] += a[i, j] / blk
    p_v, p_s = orc.block_scores(a, blk)
    assert np.allclose(p_v, pv, rtol=1e-12) and np.allclose(p_s, ps, rtol=1e-12)


# ------------------------------------------------------------------ O4 noise floor (Eq. 3-4)
def load_toy():
    p, sets, r, mu = None, {}, None, None
    with open(os.path.join(GOLDEN, "noise_floor_toy.txt")) as f:
        for line in f:
            tok = line.split()
            if not tok or tok[0] == "#":
                continue
            if tok[0] == "p":
                p = np.array([float(x) for x in tok[1:]])
            elif tok[0] == "r":
                r = float(tok[1])
            elif tok[0] == "mu":
                mu = float(tok[1])
            elif tok[0] == "alpha":
                sets[float(tok[1])] = [int(x) for x in tok[3:]]
    return p, r, mu, sets


def test_noise_floor_hand_worked_example():
    p, r, mu, sets = load_toy()
    got_r, got_mu = orc.noise_floor(p)
    assert np.isclose(got_r, r, rtol=1e-12) and np.isclose(got_mu, mu, rtol=1e-12)
    for alpha, want in sets.items():
        s, k_d, raw = orc.select_noise_floor(p, alpha, k_min=0)
        assert list(s) == want and k_d == raw == len(want)


def test_median_floor_hand_worked_example_and_properties():
    """Appendix H: the floor is the median of the non-retained blocks."""
    p = None
    sets = {}
    with open(os.path.join(GOLDEN, "noise_floor_toy.txt")) as f:
        for line in f:
            tok = line.split()
            if tok and tok[0] == "p":
                p = np.array([float(x) for x in tok[1:]])
            elif tok and tok[0] == "median_alpha":
                sets[float(tok[1])] = [int(x) for x in tok[3:]]
    assert len(sets) == 3
    for alpha, want in sets.items():
        s, k_d, raw = orc.select_median_floor(p, alpha, k_min=0)
        assert list(s) == want and k_d == raw == len(want)
    # a single dominant middle block lifts the mean floor above weaker signal but not the median floor
    q = np.array([0.5, 0.3, 0.004, 0.004, 0.004, 0.001, 0.001, 0.001, 0.001, 0.184])
    mean_set = set(orc.select_noise_floor(q, 1.0, 0)[0])
    med_set = set(orc.select_median_floor(q, 1.0, 0)[0])
    assert mean_set == {0, 1, 9} and med_set == {0, 1, 2, 3, 4, 9}
    # odd and even numbers of middle blocks; monotone in alpha; k_min fill
    r_ = rng(21)
    for nb in (7, 8, 33):
        x = r_.dirichlet(np.ones(nb) * 0.4)
        srt = np.sort(x[1:-1])
        med = srt[(nb - 2) // 2] if (nb - 2) % 2 else 0.5 * (srt[(nb - 2) // 2 - 1] + srt[(nb - 2) // 2])
        s1 = set(orc.select_median_floor(x, 1.0, 0)[0])
        assert s1 == set(np.nonzero(x > med)[0])
        assert set(orc.select_median_floor(x, 2.0, 0)[0]) <= s1 <= set(orc.select_median_floor(x, 0.5, 0)[0])
        assert orc.select_median_floor(x, 1e9, 3)[1] == 3


def test_noise_floor_literal_formula():
    """r = max(1 - p[0] - p[N_b-1], 0) as printed in Algorithm 3 line 6."""
    r_ = rng(6)
    for _ in range(20):
        p = r_.dirichlet(np.ones(12))
        got, mu = orc.noise_floor(p)
        assert np.isclose(got, max(1 - p[0] - p[-1], 0.0), rtol=1e-11, atol=1e-15)
        assert np.isclose(mu, got / 10, rtol=1e-15)


def test_noise_floor_topk_equals_threshold_set_when_unclipped():
    r_ = rng(7)
    for _ in range(50):
        nb = int(r_.integers(4, 40))
        p = r_.dirichlet(np.ones(nb) * 0.3)
        alpha = float(r_.uniform(0.2, 3.0))
        s, k_d, raw = orc.select_noise_floor(p, alpha, k_min=0)
        _, mu = orc.noise_floor(p)
        assert set(s) == set(np.nonzero(p > alpha * mu)[0])
        assert k_d == raw


def test_noise_floor_alpha_monotone_and_limits():
    r_ = rng(8)
    for _ in range(20):
        nb = 32
        p = r_.dirichlet(np.ones(nb) * 0.2)
        prev = None
        for alpha in (0.25, 0.5, 1.0, 2.0, 4.0):
            s = set(orc.select_noise_floor(p, alpha, k_min=4)[0])
            if prev is not None:
                assert s <= prev
            prev = s
        s0 = set(orc.select_noise_floor(p, 0.0, k_min=0)[0])
        assert s0 == set(np.nonzero(p > 0)[0])
        s_inf, k_d, raw = orc.select_noise_floor(p, 1e12, k_min=4)
        assert raw == 0 and k_d == 4
        assert set(s_inf) == set(np.argsort(-p, kind="stable")[:4])


def test_noise_floor_clip_to_nb():
    p = np.full(6, 1 / 6)
    s, k_d, raw = orc.select_noise_floor(p, 0.5, k_min=100)
    assert k_d == 6 and list(s) == list(range(6))


def test_noise_floor_is_sink_aware():
    """Section 4.3: growing the sink lowers mu; the selected middle set is unchanged."""
    r_ = rng(9)
    mid = r_.dirichlet(np.ones(30) * 0.3)
    base = None
    for sink in (0.1, 0.5, 0.9, 0.999):
        rest = 1.0 - sink - 0.0005
        p = np.concatenate(([sink], mid * rest, [0.0005]))
        s, _, _ = orc.select_noise_floor(p, 1.0, k_min=0)
        middle = {int(x) for x in s if 0 < x < 31}
        if base is None:
            base = middle
        assert middle == base
        r, mu = orc.noise_floor(p)
        unselected = p[[j for j in range(32) if j not in set(s)]].sum()
        assert unselected <= 1.0 * r + 1e-15


def test_stable_topk_ties_prefer_lower_index():
    p = np.array([0.1, 0.3, 0.3, 0.1, 0.2])
    assert list(orc.stable_topk(p, 1)) == [1]
    assert list(orc.stable_topk(p, 4)) == [1, 2, 4, 0]


# ------------------------------------------------------------------ O4' gamma (Algorithm 6)
def test_gamma_failure_modes_hand_worked():
    with open(os.path.join(GOLDEN, "gamma_failure_modes.txt")) as f:
        lines = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for tok in lines:
        if tok[0] == "collapse":
            gi = tok.index("gamma")
            p = np.array([float(x) for x in tok[2:gi]])
            gamma, raw = float(tok[gi + 1]), int(tok[gi + 3])
            s, k_d, got = orc.select_gamma(p, gamma, k_min=0)
            assert got == raw and list(s) == [0]
            s, k_d, got = orc.select_gamma(p, gamma, k_min=3)
            assert k_d == 3 and list(s) == [0, 1, 2]
        elif tok[0] == "residual":
            v = {tok[i]: float(tok[i + 1]) for i in range(1, len(tok), 2)}
            nbg = int(v["n_background"])
            p = np.concatenate(([v["sink"], v["signal"]], np.full(nbg, v["background"])))
            s, k_d, got = orc.select_gamma(p, v["gamma"], k_min=0)
            assert got == int(v["raw"])
            assert list(s) == list(range(int(v["raw"])))      # ties -> lower index


def test_gamma_residual_scales_linearly_with_n():
    """Appendix C: N_garbage ~ gamma_residual * n for background mass ~ 1/n."""
    counts = []
    for nb in (256, 512, 1024):
        p = np.concatenate(([0.5, 0.2], np.full(nb - 2, 0.3 / (nb - 2))))
        counts.append(orc.select_gamma(p, 0.95, 0)[2] - 2)
    for nb, c in zip((256, 512, 1024), counts):
        assert abs(c - (0.25 / 0.3) * (nb - 2)) <= 1.0


def test_gamma_limits_and_minimality():
    r_ = rng(10)
    for _ in range(20):
        p = r_.dirichlet(np.ones(24) * 0.4)
        assert orc.select_gamma(p, 1e-9, 0)[2] == 1
        assert list(orc.select_gamma(p, 1e-9, 0)[0]) == [int(np.argmax(p))]
        assert orc.select_gamma(p, 2.0, 0)[2] == 24          # never reached -> everything
        s, _, raw = orc.select_gamma(p, 0.9, 0)
        assert p[s].sum() >= 0.9
        smallest = s[np.argmin(p[s])]
        assert p[s].sum() - p[smallest] < 0.9


# ------------------------------------------------------------------ O5 PE (Algorithm 4)
def test_pooled_map_zero_inputs_closed_form():
    nb, d = 6, 4
    n = nb * B
    a = orc.pooled_map(np.zeros((n, d)), np.zeros((n, d)), B)
    for m in range(nb):
        assert np.allclose(a[m, :m + 1], 1.0 / (m + 1))
        assert np.all(a[m, m + 1:] == 0)
    sel, cut = orc.select_pe(a, 0.5)
    # entries of row m are 1/((m+1) N_b); sorted descending = rows in order; mass per row 1/N_b
    # gamma = 0.5 with N_b = 6 -> rows 0,1,2 exactly (mass 3/6), up to rounding of the cumsum
    picked_rows = [m for m in range(nb) if sel[m, :m + 1].all()]
    assert picked_rows[:3] == [0, 1, 2]
    assert sel.sum() in (6, 7)                               # 1+2+3 (+1 if 0.5 missed by an ulp)
    if sel.sum() == 7:
        assert sel[3, 0] and not sel[3, 1:].any()             # the extra entry is the first of row 3
    assert not sel[4:].any()


def test_select_pe_tie_order_is_lower_flat_index_first():
    """Algorithm 4 on a map whose entries are powers of two, so every running sum is exact.

    Normalised entries: (0,0) = 1/4; (1,0), (1,1), (2,0) = 1/8; the other six = 1/16.  Descending order with
    ties to the lower flat index m * N_b + J: (0,0) | (1,0) (1,1) (2,0) | (2,1) (2,2) (3,0) (3,1) (3,2) (3,3),
    running sums 1/4, 3/8, 1/2, 5/8, 11/16, 3/4, ...  gamma = 1/2 ends INSIDE the run of 1/8s after two of
    its three members; gamma = 0.7 ends inside the run of 1/16s after two of its six.
    """
    a = np.zeros((4, 4))
    a[0, :1] = [1.0]
    a[1, :2] = [0.5, 0.5]
    a[2, :3] = [0.5, 0.25, 0.25]
    a[3, :4] = [0.25, 0.25, 0.25, 0.25]
    sel, cut = orc.select_pe(a, 0.5)
    assert sorted(map(tuple, np.argwhere(sel).tolist())) == [(0, 0), (1, 0), (1, 1)]   # (2,0) ties but comes later
    assert cut == 0.125
    sel, cut = orc.select_pe(a, 0.7)
    assert sorted(map(tuple, np.argwhere(sel).tolist())) == [(0, 0), (1, 0), (1, 1), (2, 0), (2, 1), (2, 2)]
    assert cut == 0.0625
    # one entry more of the same tie run as soon as gamma passes the running sum
    sel, _ = orc.select_pe(a, 0.76)
    assert sel[3, 0] and not sel[3, 1:].any() and sel.sum() == 7
    # the expansion adds the forced blocks {0, m} to rows the cut left empty
    cols = orc.expand_pe(orc.select_pe(a, 0.5)[0])
    assert [c.tolist() for c in cols] == [[0], [0, 1], [0, 2], [0, 3]]


def test_head_pipeline_two_blocks_keeps_every_causal_block():
    """N_b = 2: mu_d = r_d / (N_b - 2) is undefined, and both blocks are the always-retained first and last
    block of Algorithm 3 line 12, so every causal block is kept whatever the pattern or selector."""
    r_ = rng(31)
    n, d = 2 * B, 16
    q, k, v = r_.normal(size=(n, d)), r_.normal(size=(n, d)), r_.normal(size=(n, d))
    for force in (0, 1, 2):
        for selector in (0, 1, 2):
            res = orc.head_pipeline(q, k, block=B, sink_tokens=4, local_tokens=B, force_pattern=force,
                                    selector=selector, k_min_blocks=0, alpha=50.0, gamma=1e-6)
            assert [c.tolist() for c in res["cols"]] == [[0], [0, 1]]
            assert abs(res["p_v"].sum() - 1) < 1e-12 and abs(res["p_s"].sum() - 1) < 1e-12
            # slash offset 0 = the diagonal band of the last block, offset 1 = everything older
            a = orc.proxy_attention(q, k, B)
            band0 = sum(a[i, B + i - o] for i in range(B) for o in range(B) if B + i - o >= 0 and o <= B + i) / B
            assert abs(res["p_s"][0] - band0) < 1e-12
    # Eq. 1 over those lists is dense causal attention
    o, _ = orc.sparse_attention_head(q, k, v, res["cols"], B)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q)[None, None], torch.tensor(k)[None, None], torch.tensor(v)[None, None], is_causal=True)[0, 0]
    assert np.abs(o - want.numpy()).max() < 1e-12


def test_pooled_map_bruteforce():
    nb, d, blk = 5, 3, 4
    n = nb * blk
    r = rng(11)
    q, k = r.normal(size=(n, d)), r.normal(size=(n, d))
    a = orc.pooled_map(q, k, blk)
    for m in range(nb):
        qb = [sum(q[m * blk + t, c] for t in range(blk)) / blk for c in range(d)]
        logits = []
        for J in range(m + 1):
            kb = [sum(k[J * blk + t, c] for t in range(blk)) / blk for c in range(d)]
            logits.append(sum(x * y for x, y in zip(qb, kb)) / math.sqrt(d))
        den = sum(math.exp(x - max(logits)) for x in logits)
        for J in range(m + 1):
            assert abs(a[m, J] - math.exp(logits[J] - max(logits)) / den) < 1e-14


def test_select_pe_mass_and_minimality():
    nb, d = 12, 8
    n = nb * B
    r = rng(12)
    a = orc.pooled_map(r.normal(size=(n, d)) * 3, r.normal(size=(n, d)) * 3, B)
    flat = a / a.sum()
    for gamma in (0.5, 0.9, 0.99):
        sel, cut = orc.select_pe(a, gamma)
        mass = flat[sel].sum()
        assert mass >= gamma
        assert mass - flat[sel].min() < gamma
        assert np.isclose(flat[sel].min(), cut)
        assert flat[~sel].max() <= cut
        assert not np.triu(sel, 1).any()
    assert orc.select_pe(a, 2.0)[0].sum() == nb * (nb + 1) // 2


# ------------------------------------------------------------------ O6 expansion
def token_mask_vs(s_v, s_s, nb, blk):
    n = nb * blk
    mask = np.zeros((n, n), dtype=bool)
    for t in range(n):
        for j in range(t + 1):
            m = t // blk
            if j // blk in s_v or (t - j) // blk in s_s or j // blk == 0 or j // blk == m:
                mask[t, j] = True
    return mask


def test_expand_vs_is_exact_block_cover_of_token_mask():
    r_ = rng(13)
    nb, blk = 9, 4
    for _ in range(10):
        s_v = set(int(x) for x in r_.choice(nb, size=3, replace=False))
        s_s = set(int(x) for x in r_.choice(nb, size=3, replace=False))
        cols = orc.expand_vs(sorted(s_v), sorted(s_s), nb)
        mask = token_mask_vs(s_v, s_s, nb, blk)
        for m in range(nb):
            cover = {J for J in range(m + 1)
                     if mask[m * blk:(m + 1) * blk, J * blk:(J + 1) * blk].any()}
            assert set(cols[m]) == cover
            assert list(cols[m]) == sorted(set(cols[m]))
            assert cols[m][0] == 0 and cols[m][-1] == m


def test_expand_pe_contains_forced_blocks():
    nb = 7
    sel = np.zeros((nb, nb), dtype=bool)
    sel[5, 2] = sel[5, 3] = sel[6, 6] = True
    cols = orc.expand_pe(sel)
    assert list(cols[0]) == [0] and list(cols[3]) == [0, 3]
    assert list(cols[5]) == [0, 2, 3, 5] and list(cols[6]) == [0, 6]


def test_cols_to_csr_layout():
    cols = [orc.dense_cols(3), orc.dense_cols(3)]
    row_ptr, col_idx = orc.cols_to_csr(cols)
    assert row_ptr.tolist() == [[0, 1, 3, 6], [6, 7, 9, 12]]
    assert col_idx.tolist() == [0, 0, 1, 0, 1, 2] * 2


# ------------------------------------------------------------------ O7 attention (Eq. 1)
def sdpa64(q, k, v, mask=None, causal=False):
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(x))[None, None] for x in (q, k, v))
    m = None if mask is None else torch.from_numpy(mask)[None, None]
    return torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=m, is_causal=causal)[0, 0].numpy()


def test_dense_matches_library_causal_attention():
    nb, d = 6, 16
    n = nb * B
    r = rng(14)
    q, k, v = (r.normal(size=(n, d)) for _ in range(3))
    o, lse = orc.sparse_attention_head(q, k, v, orc.dense_cols(nb), B)
    assert np.allclose(o, sdpa64(q, k, v, causal=True), rtol=1e-11, atol=1e-12)
    # lse against a direct evaluation for one row
    t = n - 3
    logits = (q[t] @ k[:t + 1].T) / math.sqrt(d)
    assert np.isclose(lse[t], np.log(np.exp(logits).sum()), rtol=1e-12)


def test_sparse_matches_library_masked_attention():
    nb, d = 8, 8
    n = nb * B
    r = rng(15)
    q, k, v = (r.normal(size=(n, d)) for _ in range(3))
    cols = orc.expand_vs([2, 5], [1, 3], nb)
    mask = np.zeros((n, n), dtype=bool)
    for m in range(nb):
        for J in cols[m]:
            mask[m * B:(m + 1) * B, J * B:(J + 1) * B] = True
    mask &= np.tril(np.ones((n, n), dtype=bool))
    o, _ = orc.sparse_attention_head(q, k, v, cols, B)
    assert np.allclose(o, sdpa64(q, k, v, mask=mask), rtol=1e-11, atol=1e-12)


def test_attention_bruteforce_three_loops():
    nb, d, blk = 3, 3, 4
    n = nb * blk
    r = rng(16)
    q, k, v = (r.normal(size=(n, d)) for _ in range(3))
    cols = [np.array([0]), np.array([0, 1]), np.array([0, 2])]
    o, _ = orc.sparse_attention_head(q, k, v, cols, blk)
    for t in range(n):
        m = t // blk
        keys = [j for j in range(t + 1) if j // blk in set(cols[m].tolist())]
        w = [math.exp(sum(q[t, c] * k[j, c] for c in range(d)) / math.sqrt(d)) for j in keys]
        for c in range(d):
            want = sum(wi * v[j, c] for wi, j in zip(w, keys)) / sum(w)
            assert abs(o[t, c] - want) < 1e-13


def test_constant_values_give_constant_output():
    nb, d = 4, 8
    n = nb * B
    r = rng(17)
    q, k = r.normal(size=(n, d)), r.normal(size=(n, d))
    v = np.tile(np.arange(d, dtype=np.float64), (n, 1))
    o, _ = orc.sparse_attention_head(q, k, v, orc.expand_vs([1], [0], nb), B)
    assert np.allclose(o, v, rtol=1e-13)


# ------------------------------------------------------------------ Algorithm 1 end to end
def test_head_pipeline_invariants_on_synthetic_heads():
    from workloads import synth
    w = synth.tiny(n=2048)
    q, k, _ = synth.make_qkv(w)
    qf, kf = q.float().numpy(), k.float().numpy()
    res = orc.layer_pipeline(qf, kf, block=128, sink_tokens=w.sink_tokens,
                             local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha,
                             gamma=w.gamma, k_min_blocks=w.k_min_blocks)
    nb = w.n_blocks
    assert [r["pattern"] for r in res] == [orc.VS, orc.VS, orc.PE, orc.PE]
    for r in res:
        assert np.isclose(r["p_v"].sum(), 1) and np.isclose(r["p_s"].sum(), 1)
        for m, cols in enumerate(r["cols"]):
            assert cols[0] == 0 and cols[-1] == m and np.all(np.diff(cols) > 0)
    # alpha monotonicity of the final lists on a VS head
    lists = {}
    for alpha in (0.5, 1.0, 2.0):
        rr = orc.head_pipeline(qf[:, 0], kf[:, 0], sink_tokens=4, tau=0.1, alpha=alpha)
        lists[alpha] = rr["cols"]
    for m in range(nb):
        assert set(lists[2.0][m]) <= set(lists[1.0][m]) <= set(lists[0.5][m])


# ------------------------------------------------------------------ Algorithm 5 (comparison router)
def test_js_distance_hand_worked_and_limits():
    """Hand-worked: a = (1, 0), b = (1/2, 1/2): m = (3/4, 1/4);
    KL(a||m) = ln(4/3), KL(b||m) = 1/2 ln(2/3) + 1/2 ln 2 -> D = sqrt(0.5 * 0.2876821 + 0.5 * 0.1438410)."""
    d = orc.js_distance(np.array([1.0, 0.0]), np.array([0.5, 0.5]))
    assert np.isclose(d, math.sqrt(0.5 * math.log(4 / 3) + 0.5 * (0.5 * math.log(2 / 3) + 0.5 * math.log(2))), rtol=1e-12)
    assert np.isclose(d, 0.4645014, rtol=1e-6)
    r_ = rng(30)
    a = r_.dirichlet(np.ones(16)); b = r_.dirichlet(np.ones(16))
    assert orc.js_distance(a, a) == 0.0
    assert np.isclose(orc.js_distance(a, b), orc.js_distance(b, a), rtol=1e-13)
    # disjoint supports: the distance reaches its maximum sqrt(ln 2)
    assert np.isclose(orc.js_distance(np.array([0.5, 0.5, 0, 0]), np.array([0, 0, 0.3, 0.7])), math.sqrt(math.log(2)), rtol=1e-13)
    assert 0.0 < orc.js_distance(a, b) < math.sqrt(math.log(2))


def test_jsd_router_closed_forms():
    """Q = 0: both estimates are known in closed form (uniform pooled estimate, uniform proxy rows)."""
    nb, d = 6, 8
    n = nb * B
    k = rng(31).normal(size=(n, d))
    dist, a_bar, a_hat = orc.jsd_router(np.zeros((n, d)), k, B)
    assert np.allclose(a_bar, 1.0 / nb)
    # a_hat[J] = (1/B) sum_i (keys of block J visible to row i) / (t_i + 1)
    want = np.zeros(nb)
    for i in range(B):
        t = n - B + i
        for J in range(nb):
            want[J] += min(max(t + 1 - J * B, 0), B) / (t + 1) / B
    assert np.allclose(a_hat, want, rtol=1e-12)
    assert np.isclose(dist, orc.js_distance(want, np.full(nb, 1 / nb)), rtol=1e-12)
    # a head whose queries all point at one key block: the pooled estimate and the per-query mean agree
    q = np.zeros((n, d)); q[:, 0] = 8.0
    k2 = np.zeros((n, d)); k2[2 * B:3 * B, 0] = 8.0
    dist2, a_bar2, a_hat2 = orc.jsd_router(q, k2, B)
    assert a_bar2[2] > 0.999 and a_hat2[2] > 0.999 and dist2 < 0.05


# ------------------------------------------------------------------ ragged n: N_b = ceil(n / B) (Section 4.3)
def test_ragged_length_block_scores_bruteforce_and_unit_mass():
    n, d, blk = 53, 4, 8              # 7 blocks, the last one holds 5 tokens
    r = rng(40)
    a = orc.proxy_attention(r.normal(size=(n, d)), r.normal(size=(n, d)), blk)
    nb = 7
    pv = [0.0] * nb
    ps = [0.0] * nb
    for i in range(blk):
        t = n - blk + i
        for j in range(t + 1):
            pv[j // blk] += a[i, j] / blk
            ps[(t - j) // blk] += a[i, j] / blk
    p_v, p_s = orc.block_scores(a, blk)
    assert p_v.shape == p_s.shape == (nb,)
    assert np.allclose(p_v, pv, rtol=1e-12) and np.allclose(p_s, ps, rtol=1e-12)
    assert np.isclose(p_v.sum(), 1) and np.isclose(p_s.sum(), 1)


def test_ragged_length_attention_matches_library():
    d = 8
    n = 5 * B + 7
    r = rng(41)
    q, k, v = (r.normal(size=(n, d)) for _ in range(3))
    nb = 6
    o, _ = orc.sparse_attention_head(q, k, v, orc.dense_cols(nb), B)
    assert np.allclose(o, sdpa64(q, k, v, causal=True), rtol=1e-11, atol=1e-12)
    cols = orc.expand_vs([2], [1], nb)
    mask = np.zeros((n, n), dtype=bool)
    for m in range(nb):
        for J in cols[m]:
            mask[m * B:(m + 1) * B, J * B:(J + 1) * B] = True
    mask &= np.tril(np.ones((n, n), dtype=bool))
    o2, _ = orc.sparse_attention_head(q, k, v, cols, B)
    assert np.allclose(o2, sdpa64(q, k, v, mask=mask), rtol=1e-11, atol=1e-12)


def test_ragged_length_pooling_and_pipeline():
    d = 8
    n = 4 * B + 3
    r = rng(42)
    x = r.normal(size=(n, d))
    bm = orc.block_means(x, B)
    assert bm.shape == (5, d)
    assert np.allclose(bm[4], x[4 * B:].mean(axis=0)) and np.allclose(bm[1], x[B:2 * B].mean(axis=0))
    res = orc.head_pipeline(x * 2, r.normal(size=(n, d)) * 2, block=B, sink_tokens=4, local_tokens=B, tau=0.0,
                            k_min_blocks=1)
    assert len(res["cols"]) == 5 and res["p_v"].shape == (5,)
    for m, c in enumerate(res["cols"]):
        assert c[0] == 0 and c[-1] == m
    res = orc.head_pipeline(np.zeros((n, d)), np.zeros((n, d)), block=B, tau=2.0, gamma=0.5)
    assert res["pattern"] == orc.PE and res["a_bar"].shape == (5, 5)
