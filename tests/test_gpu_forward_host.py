"""crisp_forward_host: Algorithm 1 on host buffers, cut into chunks of whole KV groups whose copies overlap the
kernels.  Algorithm 1 is per head, so every chunking must reproduce crisp_forward on the whole layer bit for bit."""
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B
from workloads import synth

pytestmark = pytest.mark.gpu


def _whole_layer(p, q, k, v):
    layer = crisp.CrispLayer(p)
    layer.forward(q, k, v)
    layer.poll()
    return layer.o.cpu(), layer.pattern.cpu(), int(layer.nnz.item())


@pytest.mark.parametrize("gpc", [1, 2, 4])
def test_forward_host_equals_forward_for_every_chunking(gpc):
    w = synth.llama_shaped("host", 2048 + 256, 16).with_(n_q_heads=8, n_kv_heads=4, k_min_blocks=2,
                                                       head_classes=tuple(("conc", "diffuse")[h % 2] for h in range(8)))
    p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens, local_tokens=w.local_tokens,
                          k_min_blocks=w.k_min_blocks, tau=w.tau)
    q, k, v = synth.make_qkv(w, device="cuda")
    o_ref, pat_ref, nnz_ref = _whole_layer(p, q, k, v)
    qh, kh, vh = (t.cpu().pin_memory() for t in (q, k, v))
    oh = torch.full(o_ref.shape, 7.0, dtype=o_ref.dtype).pin_memory()
    pat = torch.full((w.n_q_heads,), -1, dtype=torch.int32)
    stage = torch.empty(B.crisp_forward_host_stage_bytes(p, gpc), dtype=torch.uint8, device="cuda")
    rc, nnz = B.crisp_forward_host(p, qh, kh, vh, oh, gpc, stage, pattern_host=pat)
    assert rc == B.OK
    assert torch.equal(oh, o_ref)
    assert torch.equal(pat, pat_ref)
    assert nnz == nnz_ref
    # pageable host memory works too
    oh2 = torch.zeros_like(o_ref)
    rc, _ = B.crisp_forward_host(p, q.cpu(), k.cpu(), v.cpu(), oh2, gpc, stage)
    assert rc == B.OK and torch.equal(oh2, o_ref)


def test_forward_host_ragged_length_and_group_of_seven():
    """A length that is not a multiple of the block and the Qwen-like group size (7 query heads per KV head)."""
    n, hq, hkv = 1536 + 37, 14, 2
    q, k, v = synth.random_qkv(n, hq, hkv, seed=9, device="cuda")
    p = crisp.make_params(n, hq, hkv, sink_tokens=4, tau=0.05, k_min_blocks=2)
    o_ref, pat_ref, nnz_ref = _whole_layer(p, q, k, v)
    oh = torch.zeros_like(o_ref).pin_memory()
    pat = torch.full((hq,), -1, dtype=torch.int32)
    stage = torch.empty(B.crisp_forward_host_stage_bytes(p, 1), dtype=torch.uint8, device="cuda")
    rc, nnz = B.crisp_forward_host(p, q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory(), oh, 1, stage,
                                   pattern_host=pat)
    assert rc == B.OK and torch.equal(oh, o_ref) and torch.equal(pat, pat_ref) and nnz == nnz_ref


def test_forward_host_argument_checks():
    p = crisp.make_params(1024, 4, 2, sink_tokens=4, k_min_blocks=2)
    assert B.crisp_forward_host_stage_bytes(p, 3) == 0          # not a divisor of H_kv
    assert B.crisp_forward_host_stage_bytes(p, 0) == 0
    need = B.crisp_forward_host_stage_bytes(p, 1)
    assert need > 0
    q, k, v = synth.random_qkv(1024, 4, 2, seed=1, device="cpu")
    o = torch.empty_like(q)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    rc, _ = B.crisp_forward_host(p, q, k, v, o, 1, small)
    assert rc == B.ERR_WORKSPACE
    stage = torch.empty(need, dtype=torch.uint8, device="cuda")
    rc, _ = B.crisp_forward_host(p, q, k, v, o, 3, stage)
    assert rc == B.ERR_INVALID_ARG
