"""GPU parity: every stage of the CUDA path against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import crisp_oracle as orc
from workloads import synth

pytestmark = pytest.mark.gpu


def _pu():
    from tests import parity_utils
    return parity_utils


def _full_check(w, p=None, per_head=6, dense=True, seed=0):
    pu = _pu()
    p = p or pu.params_of(w)
    q, k, v = synth.make_qkv(w, device="cuda")
    g = pu.run_gpu(p, q, k, v, dense=dense)
    qc, kc, vc = q.cpu(), k.cpu(), v.cpu()
    res = orc.layer_pipeline(qc.float().numpy(), kc.float().numpy(), **pu.oracle_kwargs(p))
    n_lab = pu.check_route(g, res, p)
    n_exc = pu.check_lists(g, res, p)
    nb = w.n_blocks
    samples = pu.sample_blocks(nb, w.n_q_heads, per_head, seed)
    rel, mab = pu.check_attention(g, qc, kc, vc, p, samples)
    if dense:
        pu.check_attention(g, qc, kc, vc, p, samples, key="o_dense", dense=True)
    print(f"{w.name}: excused labels {n_lab}, excused blocks {n_exc}, nnz {g['nnz']}, "
          f"rel-L2 {rel:.2e}, max-abs {mab:.2e}")
    return g, res


def test_tiny_config_full():
    w = synth.CONFIGS["Tiny"]
    g, res = _full_check(w, per_head=32)
    assert [int(x) for x in g["pattern"]] == [1, 1, 0, 0]


def test_tiny_every_block_dense_and_sparse():
    pu = _pu()
    w = synth.tiny(n=2048)
    p = pu.params_of(w)
    q, k, v = synth.make_qkv(w, device="cuda")
    g = pu.run_gpu(p, q, k, v, dense=True)
    samples = [(h, m) for h in range(4) for m in range(w.n_blocks)]
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples)
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples, key="o_dense", dense=True)


@pytest.mark.parametrize("n", [256, 384, 640, 1152])
def test_small_and_odd_block_counts(n):
    """N_b = 2 (everything kept), odd N_b (a lone last tile), N_b not a multiple of the tile pair."""
    pu = _pu()
    w = synth.tiny(n=n).with_(k_min_blocks=2)
    _full_check(w, per_head=16)


@pytest.mark.parametrize("n", [257, 300, 1000, 4096 + 37, 4096 - 1, 2048 + 64])
def test_ragged_sequence_lengths(n):
    """n not a multiple of 128: N_b = ceil(n / 128), the last block is partial (Section 4.3)."""
    pu = _pu()
    w = synth.tiny(n=n).with_(k_min_blocks=2)
    g, res = _full_check(w, per_head=64)
    np.testing.assert_allclose(g["p_v"].sum(1), 1.0, rtol=1e-5)
    np.testing.assert_allclose(g["p_s"].sum(1), 1.0, rtol=1e-5)


def test_ragged_length_gqa_and_selectors():
    pu = _pu()
    w = synth.llama_shaped("L8k-r", 8192 + 77, 32).with_(n_q_heads=8, n_kv_heads=2,
                                                        head_classes=("conc", "diffuse") * 4)
    _full_check(w, per_head=6)
    _full_check(w, p=pu.params_of(w, selector=1), per_head=2, dense=False)
    _full_check(w, p=pu.params_of(w, selector=2, sink_tokens=128), per_head=2, dense=False)


def test_paper_window_sizes_and_identity():
    """w_sink = w_local = 128: C_struct equals p_v[0] + p_v[N_b-1] (Section 4.3)."""
    pu = _pu()
    w = synth.tiny(n=4096).with_(sink_tokens=128, local_tokens=128, tau=0.2)
    g, _ = _full_check(w, per_head=4, dense=False)
    np.testing.assert_allclose(g["c_struct"], g["p_v"][:, 0] + g["p_v"][:, -1], rtol=1e-5)
    np.testing.assert_allclose(g["p_v"].sum(1), 1.0, rtol=1e-5)
    np.testing.assert_allclose(g["p_s"].sum(1), 1.0, rtol=1e-5)


def test_wide_anchor_windows():
    pu = _pu()
    w = synth.tiny(n=2048).with_(sink_tokens=300, local_tokens=200)
    _full_check(w, per_head=4, dense=False)


@pytest.mark.parametrize("alpha", [0.5, 2.0])
def test_alpha_sweep_and_monotonicity(alpha):
    pu = _pu()
    w = synth.tiny(n=4096)
    g1, _ = _full_check(w, per_head=4, dense=False)
    g2, _ = _full_check(w.with_(alpha=alpha), per_head=4, dense=False)
    a, b = (g2, g1) if alpha > 1 else (g1, g2)    # a: larger alpha
    for h in (0, 1):
        for m in range(w.n_blocks):
            assert set(pu.gpu_cols(a, h, m).tolist()) <= set(pu.gpu_cols(b, h, m).tolist())


def test_gamma_selector():
    pu = _pu()
    w = synth.tiny(n=4096)
    _full_check(w, p=pu.params_of(w, selector=1), per_head=4, dense=False)
    _full_check(w, p=pu.params_of(w, selector=1, gamma=0.5), per_head=4, dense=False)


def test_median_floor_selector():
    """selector 2: the median noise floor of Appendix H (even and odd numbers of middle blocks)."""
    pu = _pu()
    for n in (4096, 4224):
        w = synth.tiny(n=n)
        _full_check(w, p=pu.params_of(w, selector=2), per_head=4, dense=False)
    w = synth.tiny(n=4096).with_(alpha=1e6, k_min_blocks=5)
    _full_check(w, p=pu.params_of(w, selector=2), per_head=2, dense=False)


@pytest.mark.parametrize("force", [1, 2])
def test_forced_patterns(force):
    pu = _pu()
    w = synth.tiny(n=2048)
    g, _ = _full_check(w, p=pu.params_of(w, force_pattern=force), per_head=4, dense=False)
    assert (g["pattern"] == (1 if force == 1 else 0)).all()


def test_k_min_fill_and_large_alpha():
    pu = _pu()
    w = synth.tiny(n=4096).with_(alpha=1e6, k_min_blocks=5)
    g, res = _full_check(w, per_head=4, dense=False)
    assert res[0]["raw_v"] < 5 and res[0]["k_v"] == 5


def test_gqa_llama_shape_reduced():
    """32k generator recipe at a reduced length: 8 query / 2 KV heads, slash lines present."""
    w = synth.llama_shaped("L8k", 8192, 32).with_(n_q_heads=8, n_kv_heads=2,
                                                  head_classes=("conc", "diffuse") * 4)
    _full_check(w, per_head=6)


def test_qwen_shape_reduced():
    """GQA group of 7, sink scale 16 (p_v[0] ~ 1: the noise floor must not cancel)."""
    w = synth.qwen_shaped("Q8k", 8192).with_(n_q_heads=14, n_kv_heads=2,
                                             head_classes=("sink", "slash", "diffuse", "diffuse") * 3
                                             + ("sink", "slash"))
    _full_check(w, per_head=4)


@pytest.mark.parametrize("hq,hkv", [(3, 3), (4, 2), (6, 2), (5, 1), (9, 1), (16, 1)])
def test_group_sizes(hq, hkv):
    """Query heads per KV head from 1 to 16: the proxy kernel handles them in chunks of four, two reduction
    groups taking the even and the odd heads of a chunk; the attention kernel shares K/V blocks per KV head."""
    pu = _pu()
    classes = tuple(("conc", "diffuse")[h % 2] for h in range(hq))
    w = synth.llama_shaped("groups", 2048 + 128, 16).with_(n_q_heads=hq, n_kv_heads=hkv, head_classes=classes,
                                                          k_min_blocks=2)
    _full_check(w, per_head=4, dense=False)


def test_iid_inputs_custom_scale():
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    n, hq, hkv = 1024, 4, 2
    q, k, v = synth.random_qkv(n, hq, hkv, seed=3, device="cuda")
    p = crisp.make_params(n, hq, hkv, sink_tokens=4, tau=0.05, softmax_scale=0.05, k_min_blocks=2)
    g = pu.run_gpu(p, q, k, v, dense=True)
    res = orc.layer_pipeline(q.cpu().float().numpy(), k.cpu().float().numpy(), **pu.oracle_kwargs(p))
    pu.check_route(g, res, p)
    pu.check_lists(g, res, p)
    samples = [(h, m) for h in range(hq) for m in range(n // 128)]
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples)
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples, key="o_dense", dense=True)


def test_logits_growing_along_the_keys_rescale_every_half_step():
    """Eq. 1 with logits that rise by 12 log2 units every 64 keys: the running maximum of every row outgrows the
    attention kernel's lazy-rescale threshold (2^8) at every half step, so the accumulator is rescaled in
    place all the way along the row (inputs with a sink-dominated maximum never take that path)."""
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    n, hq, hkv = 2048, 4, 2
    q, k, v = synth.random_qkv(n, hq, hkv, seed=11, device="cuda")
    q = (q.float() * 0.1)
    k = (k.float() * 0.1)
    q[:, :, 0] = 4.0
    k[:, :, 0] = (24.0 * (torch.arange(n, device="cuda") // 64)).unsqueeze(1)   # exact in bf16
    q, k = q.to(torch.bfloat16), k.to(torch.bfloat16)
    p = crisp.make_params(n, hq, hkv, sink_tokens=4, k_min_blocks=2)
    g = pu.run_gpu(p, q, k, v, dense=True)
    samples = [(h, m) for h in range(hq) for m in range(n // 128)]
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples)
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples, key="o_dense", dense=True)
    assert np.isfinite(g["o"]).all() and np.isfinite(g["o_dense"]).all()


def test_zero_inputs_massive_ties():
    """Q = K = 0: every proxy row is uniform and every pooled row is flat (ties everywhere)."""
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    n, hq, hkv = 1024, 2, 1
    q = torch.zeros(n, hq, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(n, hkv, 128, dtype=torch.bfloat16, device="cuda")
    v = synth.random_qkv(n, hq, hkv, seed=5, device="cuda")[2]
    for force in (1, 2):
        p = crisp.make_params(n, hq, hkv, sink_tokens=4, force_pattern=force, gamma=0.5, k_min_blocks=2)
        g = pu.run_gpu(p, q, k, v)
        nb = n // 128
        for h in range(hq):
            for m in range(nb):
                c = pu.gpu_cols(g, h, m)
                assert c[0] == 0 and c[-1] == m and np.all(np.diff(c) > 0)
        if force == 2:
            # rows in order until half of the mass: rows 0..3 of 8 (mass 4/8), later rows only {0, m}
            for m in range(4):
                assert len(pu.gpu_cols(g, 0, m)) == m + 1
            assert len(pu.gpu_cols(g, 0, 7)) == 2
        samples = [(h, m) for h in range(hq) for m in range(nb)]
        pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples)


def test_pooled_map_with_a_few_distinct_values_keeps_its_mass():
    """Key blocks that repeat four patterns: every pooled row holds four distinct values, a few hundred entries
    each, all within one binade.  The histogram levels of the gamma cut then see hundreds of entries per bin and
    CTA (their packed per-bin words must be spilled to the wide counters on the way; a build that drops the
    spilled words selects 819840 entries here instead of 766351), and an error in a bin's count or mass moves the
    cut by thousands of entries: the number of selected entries must agree with the oracle's stable-sort prefix
    to within what fp32 values against fp64 ones can shift it."""
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    nb, hq, hkv = 1280, 2, 1
    n = nb * 128
    gen = torch.Generator().manual_seed(11)
    u = torch.randn(128, generator=gen)
    u = u / u.norm()
    levels = torch.tensor([0.0, 0.1, 0.2, 0.3])           # a row's values lie within a factor e^0.3: one binade
    kb = (levels[torch.arange(nb) % 4] * 128 ** 0.5)[:, None] * u[None, :]          # [nb, 128]
    k = kb[:, None, :].expand(nb, 128, 128).reshape(n, 1, 128).to(torch.bfloat16).cuda().contiguous()
    q = u[None, None, :].expand(n, hq, 128).to(torch.bfloat16).cuda().contiguous()
    v = synth.random_qkv(n, hq, hkv, seed=6, device="cuda")[2]
    # gamma high enough for the cut to lie below the long rows, whose bins are the crowded ones: their mass counts
    p = crisp.make_params(n, hq, hkv, sink_tokens=4, force_pattern=2, gamma=0.97, k_min_blocks=2)
    layer = crisp.CrispLayer(p)
    layer.route(q, k)
    layer.select(q, k)
    layer.poll()
    torch.cuda.synchronize()
    rp = layer.row_ptr.cpu().numpy()
    a_bar = orc.pooled_map(q[:, 0].float().cpu().numpy(), k[:, 0].float().cpu().numpy(), 128)
    sel, _ = orc.select_pe(a_bar, 0.97)
    want = sum(len(c) for c in orc.expand_pe(sel))
    for h in range(hq):
        got = int(rp[h, nb] - rp[h, 0])
        assert abs(got - want) <= 64, (h, got, want)
    # and the lists are well-formed
    col = layer.col_idx[: int(layer.nnz.item())].cpu().numpy()
    for m in (0, 1, 2, 637, nb - 1):
        c = col[rp[0, m]:rp[0, m + 1]]
        assert c[0] == 0 and c[-1] == m and np.all(np.diff(c) > 0)


def test_capacity_overflow_is_reported():
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    from paper_2609_01925_b200 import binding as B
    w = synth.tiny(n=2048)
    p = pu.params_of(w)
    q, k, v = synth.make_qkv(w, device="cuda")
    layer = crisp.CrispLayer(p, capacity=10)
    layer.col_idx.fill_(-7)
    layer.route(q, k)
    layer.select(q, k)
    rc = B.crisp_poll_device_status(layer.select_ws)
    assert rc == B.ERR_CAPACITY
    assert int(layer.nnz.item()) > 10
    assert (layer.col_idx == -7).all()
    assert B.crisp_poll_device_status(layer.select_ws) == B.OK   # cleared by the poll


def test_results_are_reproducible():
    pu = _pu()
    w = synth.tiny(n=2048)
    p = pu.params_of(w)
    q, k, v = synth.make_qkv(w, device="cuda")
    a = pu.run_gpu(p, q, k, v)
    b = pu.run_gpu(p, q, k, v)
    for key in ("c_struct", "p_v", "p_s", "row_ptr", "col_idx", "o"):
        assert np.array_equal(a[key], b[key]), key


def test_jsd_comparison_router():
    """Algorithm 5 on the GPU against the oracle, and the agreement of the two routers on synthetic heads."""
    pu = _pu()
    import paper_2609_01925_b200 as crisp
    from paper_2609_01925_b200 import binding as B
    cases = [synth.tiny(n=4096),
             synth.qwen_shaped("Q8k", 8192).with_(n_q_heads=14, n_kv_heads=2,
                                                  head_classes=("sink", "slash", "diffuse", "diffuse") * 3 + ("sink", "slash"))]
    for w in cases:
        p = pu.params_of(w)
        q, k, v = synth.make_qkv(w, device="cuda")
        layer = crisp.CrispLayer(p)
        layer.route(q, k)
        jsd = torch.full((w.n_q_heads,), -1.0, device="cuda")
        pat = torch.full((w.n_q_heads,), -1, dtype=torch.int32, device="cuda")
        tau_jsd = 0.1
        B.check(B.crisp_route_jsd(p, q, k, layer.p_v, layer.select_ws, tau_jsd, jsd, pat), "crisp_route_jsd")
        torch.cuda.synchronize()
        assert B.crisp_poll_device_status(layer.select_ws) == B.OK
        qc, kc = q.cpu().float().numpy(), k.cpu().float().numpy()
        agree = 0
        for h in range(w.n_q_heads):
            want, _, _ = orc.jsd_router(qc[:, h], kc[:, h // w.group], 128)
            got = float(jsd[h].item())
            assert abs(got - want) <= 2e-4 + 2e-3 * want, (h, got, want)
            if abs(want - tau_jsd) > 1e-3 * tau_jsd:
                assert int(pat[h].item()) == (1 if want >= tau_jsd else 0)
            agree += int(pat[h].item()) == int(layer.pattern[h].item())
        print(f"{w.name}: JSD {jsd.cpu().numpy().round(3).tolist()}; C_struct and JSD routers agree on "
              f"{agree}/{w.n_q_heads} heads")
