"""The oracle pool of tests/parity_utils.py on CPU: lists and outputs that ARE the oracle's pass, a list with
one extra block and an output with one wrong element are caught.  (No GPU: the 'GPU results' are built
from the oracle here, so this covers the host logic of the full-size parity tests only.)"""
import numpy as np
import pytest
import torch

from oracle import crisp_oracle as orc
from workloads import synth

crisp = pytest.importorskip("paper_2609_01925_b200")


def _fake_gpu_results(w, p, q, k, v, pu):
    qf, kf = q.float().numpy(), k.float().numpy()
    res = orc.layer_pipeline(qf, kf, **pu.oracle_kwargs(p))
    row_ptr, col_idx = orc.cols_to_csr([r["cols"] for r in res])
    g = dict(c_struct=np.array([r["c_struct"] for r in res], np.float32),
             pattern=np.array([r["pattern"] for r in res], np.int32),
             p_v=np.stack([r["p_v"] for r in res]).astype(np.float32),
             p_s=np.stack([r["p_s"] for r in res]).astype(np.float32),
             row_ptr=row_ptr, col_idx=col_idx, nnz=int(col_idx.shape[0]))
    return g, res


def test_pool_accepts_oracle_results_and_catches_planted_errors():
    from tests import parity_utils as pu
    w = synth.tiny(n=4096)
    q, k, v = synth.make_qkv(w, device="cpu")
    p = pu.params_of(w)
    g, res = _fake_gpu_results(w, p, q, k, v, pu)
    hq, nb = w.n_q_heads, w.n_blocks
    vf = v.float().numpy()

    def fetch(h, m):
        cols = pu.gpu_cols(g, h, m)
        o, _ = orc.sparse_attention_block(q[:, h].float().numpy(), k[:, 0].float().numpy(), vf[:, 0], m, cols, 128)
        return o.astype(np.float32)

    samples = pu.sample_blocks(nb, hq, 4, seed=1)
    with pu.OraclePool(p, q, k, v, g, workers=2) as pool:
        small, labels, exc = pool.heads(g, list(range(hq)), band_limit=1.0)   # 32 blocks: two in the band are 3 %
        assert labels == 0 and set(exc.per_head) == set(range(hq))
        assert [r["pattern"] for r in small] == [r["pattern"] for r in res]
        rel, mab, blocks = pool.attention(g, samples, fetch)
        assert rel < 1e-6 and blocks == sum(len(pu.gpu_cols(g, h, m)) for h, m in samples)
        with pytest.raises(AssertionError):
            pool.attention(g, samples[:2], lambda h, m: fetch(h, m) + 0.05)
    # one block too many in a row of a VS head: rebuild the lists with it and expect "extra"
    h = int(np.nonzero(g["pattern"] == orc.VS)[0][0])
    cols = [list(c) for c in res[h]["cols"]]
    m = nb - 1
    missing_block = next(j for j in range(1, m) if j not in cols[m])
    cols[m] = sorted(cols[m] + [missing_block])
    lists = [r["cols"] for r in res]
    lists[h] = [np.asarray(c, np.int32) for c in cols]
    g2 = dict(g)
    g2["row_ptr"], g2["col_idx"] = orc.cols_to_csr(lists)
    with pu.OraclePool(p, q, k, v, g2, workers=2) as pool:
        with pytest.raises(AssertionError, match="extra"):
            pool.heads(g2, [h], band_limit=1.0)
