"""crisp_forward: Algorithm 1 in one call, the context-length gate, and the device-side guard that
keeps the attention kernels away from lists that did not fit their capacity."""
import numpy as np
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B
from workloads import synth

pytestmark = pytest.mark.gpu


def _setup(n=2048, **kw):
    w = synth.tiny(n=n)
    q, k, v = synth.make_qkv(w, device="cuda")
    p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens,
                          local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha, gamma=w.gamma)
    return w, p, q, k, v


def test_forward_equals_the_staged_calls():
    w, p, q, k, v = _setup()
    a = crisp.CrispLayer(p, with_lse=True)
    a.route(q, k); a.select(q, k); a.sparse_prefill(q, k, v); a.poll()
    b = crisp.CrispLayer(p, with_lse=True)
    b.forward(q, k, v); b.poll()
    torch.cuda.synchronize()
    nnz = int(a.nnz.item())
    assert int(b.nnz.item()) == nnz
    for x, y in ((a.o, b.o), (a.lse, b.lse), (a.row_ptr, b.row_ptr), (a.col_idx[:nnz], b.col_idx[:nnz]),
                 (a.pattern, b.pattern), (a.p_v, b.p_v), (a.p_s, b.p_s), (a.c_struct, b.c_struct)):
        assert torch.equal(x, y)


def test_gate_runs_the_dense_kernel_below_the_threshold():
    w, p, q, k, v = _setup()
    a = crisp.CrispLayer(p)
    a.dense_prefill(q, k, v); a.poll()
    b = crisp.CrispLayer(p)
    b.pattern.fill_(-5); b.nnz.fill_(-5)
    b.forward(q, k, v, dense_below_tokens=w.seq_len + 1); b.poll()
    torch.cuda.synchronize()
    assert torch.equal(a.o, b.o)
    assert (b.pattern == -5).all() and int(b.nnz.item()) == -5       # routing and selection did not run
    # at the threshold itself the sparse path runs
    b.forward(q, k, v, dense_below_tokens=w.seq_len); b.poll()
    assert (b.pattern >= 0).all() and int(b.nnz.item()) > 0
    # the gated dense call needs neither the routing buffers nor their workspaces
    rc = B.load().crisp_forward(__import__("ctypes").byref(p), q.data_ptr(), k.data_ptr(), v.data_ptr(), None, 0,
                                None, 0, b.prefill_ws.data_ptr(), b.prefill_ws.numel(), None, None, None, None,
                                None, None, 0, None, b.o.data_ptr(), None, w.seq_len + 1, None)
    assert rc == B.OK
    torch.cuda.synchronize()
    assert torch.equal(a.o, b.o)


def test_lists_that_do_not_fit_are_never_read():
    w, p, q, k, v = _setup()
    layer = crisp.CrispLayer(p, capacity=16)
    layer.col_idx.fill_(0x7fffffff)            # would index far out of bounds if it were read
    layer.o.fill_(7.0)
    layer.forward(q, k, v)
    torch.cuda.synchronize()
    assert B.crisp_poll_device_status(layer.select_ws) == B.ERR_CAPACITY
    assert B.crisp_poll_device_status(layer.prefill_ws) == B.OK
    assert (layer.o == 7.0).all()                # attention did nothing
    assert (layer.col_idx == 0x7fffffff).all()
    assert int(layer.nnz.item()) > 16
    # the same layer works again once the capacity is enough
    big = crisp.CrispLayer(p)
    big.forward(q, k, v); big.poll()
    assert not (big.o == 7.0).all()


def test_forward_replays_from_a_cuda_graph():
    """The staged kernels of crisp_forward contain no host synchronisation, so one capture replays the
    whole of Algorithm 1 (this is how a caller removes the per-launch host cost at short contexts)."""
    w, p, q, k, v = _setup(n=4096)
    layer = crisp.CrispLayer(p)
    layer.forward(q, k, v); layer.poll()
    torch.cuda.synchronize()
    ref = layer.o.clone()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        layer.forward(q, k, v, stream=s)          # warm-up on the side stream
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            layer.forward(q, k, v, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    layer.o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    layer.poll()
    assert torch.equal(layer.o, ref)


def test_per_kernel_profile_records():
    """crisp_profile_enable / crisp_profile_read: one record per kernel the stage calls launch, in launch order,
    with positive device times; nothing is recorded while profiling is off."""
    w, p, q, k, v = _setup()
    layer = crisp.CrispLayer(p)
    layer.route(q, k); layer.select(q, k); layer.sparse_prefill(q, k, v); layer.poll()
    B.crisp_profile_enable(True)
    layer.route(q, k); layer.select(q, k); layer.sparse_prefill(q, k, v)
    recs = B.crisp_profile_read()
    B.crisp_profile_enable(False)
    names = [n for n, _ in recs]
    assert names[:2] == ["proxy", "tile_sums"] and names[-1] == "prefill_sparse" and "fill" in names
    # 2048 tokens take the short-prompt selection kernel and, with an SM for every attention item, no schedule
    # sort (7 launches); more than 64 blocks take 12
    assert len(names) == 7 and "pe_small" in names and "sched_scatter" not in names and "pe_rows" not in names
    assert all(ms > 0 for _, ms in recs)
    layer.route(q, k)
    assert B.crisp_profile_read() == []
    layer.poll()
