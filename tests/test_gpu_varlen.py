"""Packed batches of sequences (crisp_forward_varlen) and dense attention on lengths below two blocks.

A packed batch is defined as "every sequence processed as if it were alone", so the checks are (1) bit
equality with crisp_forward / crisp_dense_prefill on each sequence's slab, and (2) the fp64 oracle on
sequences taken out of the batch's outputs.
"""
import numpy as np
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B
from oracle import crisp_oracle as orc
from workloads import synth

pytestmark = pytest.mark.gpu

HQ, HKV = 4, 1


def _pu():
    from tests import parity_utils
    return parity_utils


def _sequence(length, seed):
    """Inputs of one sequence: the structured Tiny recipe when it can be routed, iid otherwise."""
    if length >= 256:
        return synth.make_qkv(synth.tiny(n=length, seed=seed), device="cuda")
    return synth.random_qkv(length, HQ, HKV, seed=seed, device="cuda")


def _params(n):
    w = synth.tiny(n=max(n, 256))
    return crisp.make_params(n, HQ, HKV, sink_tokens=w.sink_tokens, local_tokens=w.local_tokens, tau=w.tau,
                             alpha=w.alpha, gamma=w.gamma, k_min_blocks=2)


@pytest.mark.parametrize("n", [1, 5, 100, 128, 129, 200, 255])
def test_dense_prefill_below_two_blocks(n):
    pu = _pu()
    q, k, v = synth.random_qkv(n, HQ, HKV, seed=n, device="cuda")
    p = _params(n)
    layer = crisp.CrispLayer(p, with_lse=True)
    layer.o.fill_(7.0)
    layer.dense_prefill(q, k, v)
    B.check(B.crisp_poll_device_status(layer.prefill_ws), "dense prefill")
    torch.cuda.synchronize()
    g = dict(o_dense=layer.o.float().cpu().numpy(), lse_dense=layer.lse.cpu().numpy())
    nb = (n + 127) // 128
    samples = [(h, m) for h in range(HQ) for m in range(nb)]
    pu.check_attention(g, q.cpu(), k.cpu(), v.cpu(), p, samples, key="o_dense", dense=True)


class _Batch:
    """Device buffers of a packed batch, laid out as include/crisp.h says."""

    def __init__(self, lens, dense_below_tokens=0, capacity=None):
        self.lens = lens
        self.cu = [0]
        for x in lens:
            self.cu.append(self.cu[-1] + x)
        self.dense_below = dense_below_tokens
        parts = [_sequence(x, seed=10 + b) for b, x in enumerate(lens) if x > 0]
        self.q = torch.cat([t[0] for t in parts])
        self.k = torch.cat([t[1] for t in parts])
        self.v = torch.cat([t[2] for t in parts])
        total = self.cu[-1]
        self.p = _params(max(lens))
        rws, sws, pws = B.crisp_workspace_bytes(self.p)
        dev = "cuda"
        self.route_ws = torch.zeros(rws, dtype=torch.uint8, device=dev)
        self.select_ws = torch.zeros(sws, dtype=torch.uint8, device=dev)
        self.prefill_ws = torch.zeros(pws, dtype=torch.uint8, device=dev)
        self.nb = [(x + 127) // 128 for x in lens]
        routed_causal = sum(b * (b + 1) // 2 for x, b in zip(lens, self.nb)
                            if x >= max(256, dense_below_tokens))
        self.capacity = HQ * routed_causal if capacity is None else capacity
        self.blk_off, self.col_off = B.crisp_varlen_layout(self.p, self.cu, self.capacity, dense_below_tokens)
        nblk = self.blk_off[-1]
        batch = len(lens)
        self.c_struct = torch.full((batch, HQ), -1.0, dtype=torch.float32, device=dev)
        self.pattern = torch.full((batch, HQ), -5, dtype=torch.int32, device=dev)
        self.p_v = torch.full((HQ * nblk,), -1.0, dtype=torch.float32, device=dev)
        self.p_s = torch.full((HQ * nblk,), -1.0, dtype=torch.float32, device=dev)
        self.row_ptr = torch.full((HQ * (nblk + batch),), -1, dtype=torch.int64, device=dev)
        self.col_idx = torch.full((max(self.capacity, 1),), -1, dtype=torch.int32, device=dev)
        self.nnz = torch.full((batch,), -5, dtype=torch.int64, device=dev)
        self.status = torch.full((batch, 2), 99, dtype=torch.int32, device=dev)
        self.o = torch.full((total, HQ, 128), 7.0, dtype=torch.bfloat16, device=dev)
        self.lse = torch.full((HQ * total,), 7.0, dtype=torch.float32, device=dev)

    def run(self):
        B.check(B.crisp_forward_varlen(self.p, self.cu, self.q, self.k, self.v, self.route_ws, self.select_ws,
                                       self.prefill_ws, self.c_struct, self.pattern, self.p_v, self.p_s,
                                       self.row_ptr, self.col_idx, self.capacity, self.nnz, self.status, self.o,
                                       self.lse, self.dense_below), "crisp_forward_varlen")
        torch.cuda.synchronize()

    def routed(self, b):
        return self.lens[b] >= max(256, self.dense_below)

    def slab(self, t, b):
        return t[self.cu[b]:self.cu[b + 1]]

    def outputs(self, b):
        """The outputs of sequence b, shaped as a single-sequence call would return them."""
        n, nb = self.lens[b], self.nb[b]
        out = dict(o=self.slab(self.o, b), lse=self.lse[HQ * self.cu[b]:HQ * self.cu[b + 1]].view(HQ, n))
        if self.routed(b):
            o0 = HQ * self.blk_off[b]
            r0 = HQ * (self.blk_off[b] + b)
            nnz = int(self.nnz[b].item())
            out.update(c_struct=self.c_struct[b], pattern=self.pattern[b],
                       p_v=self.p_v[o0:o0 + HQ * nb].view(HQ, nb), p_s=self.p_s[o0:o0 + HQ * nb].view(HQ, nb),
                       row_ptr=self.row_ptr[r0:r0 + HQ * (nb + 1)].view(HQ, nb + 1), nnz=nnz,
                       col_idx=self.col_idx[self.col_off[b]:self.col_off[b] + nnz])
        return out


LENS = [300, 0, 1000, 128, 70, 2112, 257]


def test_varlen_equals_each_sequence_alone():
    bt = _Batch(LENS)
    bt.run()
    assert bt.status.cpu().tolist() == [[0, 0]] * len(LENS)
    for b, n in enumerate(LENS):
        if n == 0:
            continue
        q, k, v = (bt.slab(t, b).contiguous() for t in (bt.q, bt.k, bt.v))
        alone = crisp.CrispLayer(_params(n), with_lse=True)
        got = bt.outputs(b)
        if bt.routed(b):
            alone.forward(q, k, v)
            alone.poll()
            torch.cuda.synchronize()
            nnz = int(alone.nnz.item())
            assert got["nnz"] == nnz
            assert bt.col_off[b + 1] - bt.col_off[b] >= nnz
            for name, want in (("c_struct", alone.c_struct), ("pattern", alone.pattern), ("p_v", alone.p_v),
                               ("p_s", alone.p_s), ("row_ptr", alone.row_ptr), ("col_idx", alone.col_idx[:nnz])):
                assert torch.equal(got[name], want), (b, name)
        else:
            alone.dense_prefill(q, k, v)
            B.check(B.crisp_poll_device_status(alone.prefill_ws), "dense prefill")
            torch.cuda.synchronize()
            assert int(bt.nnz[b].item()) == -5 and (bt.pattern[b] == -5).all()    # untouched
        assert torch.equal(got["o"], alone.o), b
        assert torch.equal(got["lse"], alone.lse), b


def test_varlen_against_the_oracle():
    """Two sequences out of a batch, through the same checks as a single sequence."""
    pu = _pu()
    bt = _Batch(LENS)
    bt.run()
    for b in (2, 6):
        n = LENS[b]
        p = _params(n)
        q, k, v = (bt.slab(t, b).cpu() for t in (bt.q, bt.k, bt.v))
        got = bt.outputs(b)
        g = {key: (val.float().cpu().numpy() if key == "o" else val.cpu().numpy() if torch.is_tensor(val) else val)
             for key, val in got.items()}
        res = orc.layer_pipeline(q.float().numpy(), k.float().numpy(), **pu.oracle_kwargs(p))
        pu.check_route(g, res, p)
        pu.check_lists(g, res, p)
        samples = [(h, m) for h in range(HQ) for m in range(bt.nb[b])]
        pu.check_attention(g, q, k, v, p, samples)
    # a dense sequence of the batch (70 tokens) against the definition
    b = 4
    g = dict(o_dense=bt.outputs(b)["o"].float().cpu().numpy(), lse_dense=bt.outputs(b)["lse"].cpu().numpy())
    q, k, v = (bt.slab(t, b).cpu() for t in (bt.q, bt.k, bt.v))
    pu.check_attention(g, q, k, v, _params(LENS[b]), [(h, 0) for h in range(HQ)], key="o_dense", dense=True)


def test_varlen_gate_and_capacity():
    # the gate sends everything below 1024 tokens to dense attention
    bt = _Batch(LENS, dense_below_tokens=1024)
    bt.run()
    for b, n in enumerate(LENS):
        routed = n >= 1024
        assert bt.routed(b) == routed
        assert (int(bt.nnz[b].item()) > 0) == routed
    for b, n in enumerate(LENS):
        if 0 < n < 1024:       # dense: the same bits as the dense call on the sequence alone
            alone = crisp.CrispLayer(_params(n))
            alone.dense_prefill(*(bt.slab(t, b).contiguous() for t in (bt.q, bt.k, bt.v)))
            torch.cuda.synchronize()
            assert torch.equal(bt.outputs(b)["o"], alone.o), b
    # a share of col_idx that is too small: that sequence reports it and its rows of O stay untouched,
    # the others are unaffected
    small = _Batch(LENS, capacity=200)
    small.run()
    st = small.status.cpu().tolist()
    full = _Batch(LENS)
    full.run()
    hit = [b for b in range(len(LENS)) if st[b][0] == B.ERR_CAPACITY]
    assert hit, st
    for b, n in enumerate(LENS):
        if n == 0:
            continue
        if b in hit:
            assert (small.outputs(b)["o"] == 7.0).all()
            assert int(small.nnz[b].item()) > small.col_off[b + 1] - small.col_off[b]
        else:
            assert st[b] == [0, 0]
            assert torch.equal(small.outputs(b)["o"], full.outputs(b)["o"])


def test_varlen_rejects_bad_arguments():
    bt = _Batch([300, 400])
    rc = B.crisp_forward_varlen(bt.p, [0, 300, 700], bt.q, bt.k, bt.v, bt.route_ws[:1024], bt.select_ws, bt.prefill_ws,
                                bt.c_struct, bt.pattern, bt.p_v, bt.p_s, bt.row_ptr, bt.col_idx, bt.capacity, bt.nnz,
                                bt.status, bt.o, bt.lse)
    assert rc == B.ERR_WORKSPACE
    rc = B.crisp_forward_varlen(bt.p, [0, 300, 200], bt.q, bt.k, bt.v, bt.route_ws, bt.select_ws, bt.prefill_ws,
                                bt.c_struct, bt.pattern, bt.p_v, bt.p_s, bt.row_ptr, bt.col_idx, bt.capacity, bt.nnz,
                                bt.status, bt.o, bt.lse)
    assert rc == B.ERR_INVALID_ARG
    # an empty batch is fine and does nothing
    assert B.crisp_forward_varlen(bt.p, [0], bt.q, bt.k, bt.v, None, None, None, None, None, None, None, None, None,
                                  0, None, None, bt.o, None) == B.OK
