"""crisp_route_static: the routing stage for callers that cannot allocate device memory.

Some users of this library run inside a host program that has already taken all device memory for
its own pool, or inside a serving loop where any allocating CUDA call is forbidden; they cannot
provide the workspace crisp_route asks for.  crisp_route_static keeps that scratch in a fixed 4 MiB
array inside the library instead.  This file checks, through the C ABI, that it returns what
crisp_route returns - twice in a row, because every call reuses the same array and must not be
affected by what the previous call left in it - and that problems too large for the array are
refused on the host.  The file name makes pytest collect it after every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B
from workloads import synth


def test_static_route_refuses_problems_beyond_its_scratch():
    lib = B.load()
    p = crisp.make_params(32768, 32, 8)          # needs ~12.6 MB of scratch
    assert B.crisp_workspace_bytes(p)[0] > B.ROUTE_STATIC_SCRATCH_BYTES
    fake = ctypes.c_void_p(0x1000)               # never dereferenced: the size check comes first
    rc = lib.crisp_route_static(ctypes.byref(p), fake, fake, fake, fake, fake, fake, None, None)
    assert rc == B.ERR_UNSUPPORTED
    assert "scratch" in B.last_cuda_error() and "4194304" in B.last_cuda_error()
    small = crisp.make_params(8192, 32, 8)
    assert B.crisp_workspace_bytes(small)[0] <= B.ROUTE_STATIC_SCRATCH_BYTES
    assert lib.crisp_route_static(ctypes.byref(small), None, fake, fake, fake, fake, fake, None,
                                  None) == B.ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_route_matches_route_on_two_calls_in_a_row():
    dev = torch.device("cuda")
    cases = [synth.tiny(n=2048),
             synth.llama_shaped("L8k", 8192, 32).with_(n_q_heads=8, n_kv_heads=2,
                                                       head_classes=("conc", "diffuse") * 4),
             synth.tiny(n=2048 + 37),                      # a length that is not a multiple of the block
             synth.llama_shaped("L8k-32", 8192, 32)]       # 32 heads x 8192 tokens: just inside the 4 MiB
    for w in cases:                               # the second case reuses the array after the first
        q, k, _ = synth.make_qkv(w, device=dev)
        p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens,
                              local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha, gamma=w.gamma)
        hq, nb = w.n_q_heads, w.n_blocks
        ws = torch.zeros(B.crisp_workspace_bytes(p)[0], dtype=torch.uint8, device=dev)

        def outputs():
            return (torch.full((hq,), -1.0, device=dev), torch.full((hq,), -1, dtype=torch.int32, device=dev),
                    torch.full((hq, nb), -1.0, device=dev), torch.full((hq, nb), -1.0, device=dev))

        ref = outputs()
        B.check(B.crisp_route(p, q, k, ws, *ref), "crisp_route")
        assert B.crisp_poll_device_status(ws) == B.OK
        for call in range(2):
            got = outputs()
            status = torch.full((1,), 123, dtype=torch.int32, device=dev)
            B.check(B.crisp_route_static(p, q, k, *got, device_status=status), "crisp_route_static")
            torch.cuda.synchronize()
            assert int(status.item()) == B.OK, call
            assert torch.equal(got[1], ref[1]), (w.name, call)                     # routing labels
            for a, b in zip((got[0], got[2], got[3]), (ref[0], ref[2], ref[3])):   # C_struct, p_v, p_s
                np.testing.assert_allclose(a.cpu().numpy(), b.cpu().numpy(), rtol=2e-4, atol=1e-7)
            np.testing.assert_allclose(got[2].sum(1).cpu().numpy(), 1.0, rtol=1e-5)
