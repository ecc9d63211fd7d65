"""Failure reporting on the device without any GPU fault: index lists that break the list rules are
refused by the validating merge kernel (nothing is computed from them, O stays untouched), and a bounded
wait that runs out reports CRISP_ERR_DEVICE_TIMEOUT while the kernel returns by itself.

Every bad list used here stays inside the buffers (columns below N_b, offsets below the list size), so
even a wrong check could not make the kernels read or write out of range.
"""
import numpy as np
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B
from workloads import synth

pytestmark = pytest.mark.gpu


def _layer(n=4096):
    w = synth.tiny(n=n)
    q, k, v = synth.make_qkv(w, device="cuda")
    p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens,
                          local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha, gamma=w.gamma)
    layer = crisp.CrispLayer(p)
    layer.route(q, k); layer.select(q, k); layer.poll()
    torch.cuda.synchronize()
    return w, p, q, k, v, layer


def _run_lists(layer, p, q, k, v, row_ptr, col_idx):
    sentinel = 7.0
    layer.o.fill_(sentinel)
    B.check(B.crisp_sparse_prefill(p, q, k, v, row_ptr, col_idx, layer.prefill_ws, layer.o), "crisp_sparse_prefill")
    status = B.crisp_poll_device_status(layer.prefill_ws)
    torch.cuda.synchronize()
    untouched = bool((layer.o == sentinel).all())
    return status, untouched


def test_corrupted_lists_are_refused_and_nothing_is_computed():
    w, p, q, k, v, layer = _layer()
    nb, hq = w.n_blocks, w.n_q_heads
    rp = layer.row_ptr.clone()
    ci = layer.col_idx.clone()
    status, untouched = _run_lists(layer, p, q, k, v, rp, ci)
    assert status == B.OK and not untouched                       # the unmodified lists are fine
    good = layer.o.clone()
    rph = rp.cpu().numpy()
    cih = ci.cpu().numpy()
    # a row with at least two entries whose last-but-one column is below m - 1 (so that moving the diagonal
    # entry down to m - 1 keeps the row ascending and only removes the diagonal)
    h, m = next((h, m) for h in range(hq) for m in range(2, nb - 1)
                if rph[h, m + 1] - rph[h, m] >= 2 and cih[rph[h, m + 1] - 2] < m - 1)
    lo, hi = int(rph[h, m]), int(rph[h, m + 1])

    def corrupted(pos, value):
        c = ci.clone()
        c[pos] = value
        return c

    cases = {
        "column above the query block": corrupted(hi - 1, m + 1),   # m + 1 < N_b: still a valid block
        "diagonal missing": corrupted(hi - 1, m - 1),
        "duplicate entry": corrupted(lo + 1, int(cih[lo])),
        "negative column": corrupted(lo, -1),
    }
    for name, c in cases.items():
        status, untouched = _run_lists(layer, p, q, k, v, rp, c)
        assert status == B.ERR_BAD_LIST, name
        assert untouched, name
    # row_ptr faults: a row longer than m + 1 entries, an empty row, a decreasing offset
    for name, edit in (("row too long", lambda r: r[0, 1].__iadd__(5)),
                       ("empty row", lambda r: r[h, m + 1].copy_(r[h, m])),
                       ("decreasing", lambda r: r[h, m + 1].copy_(r[h, m] - 1))):
        r = rp.clone()
        edit(r)
        status, untouched = _run_lists(layer, p, q, k, v, r, ci)
        assert status == B.ERR_BAD_LIST, name
        assert untouched, name
    # the workspace and the context are still good: the original lists give the original result
    status, untouched = _run_lists(layer, p, q, k, v, rp, ci)
    assert status == B.OK
    assert torch.equal(layer.o, good)


def test_bounded_wait_runs_out_and_reports_timeout():
    w, p, q, k, v, layer = _layer()
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    limit_ns = 500_000                                              # 0.5 ms
    assert B.crisp_selftest_bounded_wait(ws, limit_ns) == B.OK
    assert B.crisp_poll_device_status(ws) == B.ERR_DEVICE_TIMEOUT   # the kernel has returned by itself
    waited = ws[64:80].view(torch.int64).cpu().numpy()
    assert limit_ns <= waited[0] <= 20 * limit_ns, waited           # the short wait ran to its limit
    assert waited[1] <= 50 * limit_ns, waited                       # the 400 ms wait was cut short by the abort flag
    assert B.crisp_poll_device_status(ws) == B.OK                   # polling cleared the word
    # limits outside 1 ns .. 10 ms are refused on the host
    assert B.crisp_selftest_bounded_wait(ws, 0) == B.ERR_INVALID_ARG
    assert B.crisp_selftest_bounded_wait(ws, 10_000_001) == B.ERR_INVALID_ARG
    # the context is still usable: a normal stage call runs and reports no error
    layer.sparse_prefill(q, k, v)
    layer.poll()
