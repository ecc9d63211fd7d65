"""GPU parity on randomly drawn shapes and parameters (fixed seeds): ragged lengths, GQA group sizes, forced
patterns, the three selectors, gamma and alpha away from the defaults.  Every case goes through the same checks
as the named configurations: labels, lists under the matching rule, sampled attention blocks against the oracle."""
import random

import pytest
import torch

from oracle import crisp_oracle as orc
from workloads import synth

pytestmark = pytest.mark.gpu


def _case(rng, sizes):
    return dict(n=rng.choice(sizes)(rng), seed=rng.randrange(1000), kind=rng.choice(["planted", "planted", "iid"]),
                gamma=rng.choice([0.5, 0.8, 0.95, 0.99]), alpha=rng.choice([0.5, 1.0, 2.0]),
                force=rng.choice([0, 0, 2]), selector=rng.choice([0, 0, 1, 2]),
                heads=rng.choice([(2, 1), (4, 2), (6, 2), (8, 1)]))


_SMALL = [lambda r: r.randrange(300, 3000), lambda r: r.randrange(3000, 9000), lambda r: r.randrange(9000, 20000),
          lambda r: 128 * r.randrange(3, 130)]
_LARGE = [lambda r: r.randrange(20000, 60000), lambda r: r.randrange(60000, 120000), lambda r: 128 * r.randrange(500, 900)]


def _run(c):
    from tests import parity_utils as pu
    from tests.test_gpu_parity import _full_check
    import paper_2609_01925_b200 as crisp
    if c["kind"] == "planted":
        w = synth.tiny(seed=c["seed"], n=c["n"]).with_(gamma=c["gamma"], alpha=c["alpha"])
        _full_check(w, p=pu.params_of(w, force_pattern=c["force"], selector=c["selector"]), per_head=3,
                    dense=c["seed"] % 3 == 0, seed=c["seed"])
        return
    hq, hkv = c["heads"]
    n = c["n"]
    q, k, v = synth.random_qkv(n, hq, hkv, seed=c["seed"], device="cuda")
    p = crisp.make_params(n, hq, hkv, sink_tokens=4, gamma=c["gamma"], alpha=c["alpha"], force_pattern=c["force"],
                          selector=c["selector"], k_min_blocks=2)
    g = pu.run_gpu(p, q, k, v)
    res = orc.layer_pipeline(q.cpu().float().numpy(), k.cpu().float().numpy(), **pu.oracle_kwargs(p))
    pu.check_route(g, res, p)
    pu.check_lists(g, res, p)
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, pu.sample_blocks(-(-n // 128), hq, 3, c["seed"]))


@pytest.mark.parametrize("index", range(24))
def test_random_small_cases(index):
    rng = random.Random(1000 + index)
    _run(_case(rng, _SMALL))


@pytest.mark.parametrize("index", range(6))
def test_random_large_cases(index):
    rng = random.Random(2000 + index)
    c = _case(rng, _LARGE)
    c["heads"] = (2, 1) if c["heads"][0] > 4 else c["heads"]
    _run(c)
