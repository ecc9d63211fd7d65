"""Buffer owner for one attention layer: allocates workspaces and outputs, calls the C ABI."""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


class CrispLayer:
    """Holds the device buffers of one (seq_len, heads) problem and runs the four C-ABI stages.

    Algorithm 1 of the paper = route() -> select() -> sparse_prefill().  Nothing is computed in
    Python; every method only passes pointers to libcrisp.so.
    """

    def __init__(self, params: B.CrispParams, device="cuda", capacity: Optional[int] = None,
                 with_lse: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("CrispLayer needs a CUDA device (no CPU fallback)")
        self.p = params
        self.device = torch.device(device)
        n, hq = params.seq_len, params.n_q_heads
        self.nb = -(-n // params.block)
        rws, sws, pws = B.crisp_workspace_bytes(params)
        dev = self.device
        self.route_ws = torch.empty(rws, dtype=torch.uint8, device=dev)
        self.select_ws = torch.empty(sws, dtype=torch.uint8, device=dev)
        self.prefill_ws = torch.empty(pws, dtype=torch.uint8, device=dev)
        for ws in (self.route_ws, self.select_ws, self.prefill_ws):
            ws[:256].zero_()   # status word: defined even before the first stage call
        self.c_struct = torch.empty(hq, dtype=torch.float32, device=dev)
        self.pattern = torch.empty(hq, dtype=torch.int32, device=dev)
        self.p_v = torch.empty(hq, self.nb, dtype=torch.float32, device=dev)
        self.p_s = torch.empty(hq, self.nb, dtype=torch.float32, device=dev)
        self.row_ptr = torch.empty(hq, self.nb + 1, dtype=torch.int64, device=dev)
        self.capacity = int(capacity) if capacity is not None else hq * self.nb * (self.nb + 1) // 2
        self.col_idx = torch.empty(max(self.capacity, 1), dtype=torch.int32, device=dev)
        self.nnz = torch.zeros(1, dtype=torch.int64, device=dev)
        self.o = torch.empty(n, hq, params.head_dim, dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty(hq, n, dtype=torch.float32, device=dev) if with_lse else None

    def route(self, q, k, stream=None):
        B.check(B.crisp_route(self.p, q, k, self.route_ws, self.c_struct, self.pattern, self.p_v,
                              self.p_s, stream), "crisp_route")

    def select(self, q, k, stream=None):
        B.check(B.crisp_select(self.p, q, k, self.pattern, self.p_v, self.p_s, self.select_ws,
                               self.row_ptr, self.col_idx, self.capacity, self.nnz, stream),
                "crisp_select")

    def sparse_prefill(self, q, k, v, stream=None):
        B.check(B.crisp_sparse_prefill(self.p, q, k, v, self.row_ptr, self.col_idx, self.prefill_ws,
                                       self.o, self.lse, stream), "crisp_sparse_prefill")

    def dense_prefill(self, q, k, v, stream=None):
        B.check(B.crisp_dense_prefill(self.p, q, k, v, self.prefill_ws, self.o, self.lse, stream),
                "crisp_dense_prefill")

    def forward(self, q, k, v, stream=None, dense_below_tokens: int = 0):
        """Algorithm 1 through crisp_forward (one C call: route, select, sparse attention, or the dense
        kernel when seq_len < dense_below_tokens).  Returns O [n, H_q, 128] bf16."""
        B.check(B.crisp_forward(self.p, q, k, v, self.route_ws, self.select_ws, self.prefill_ws, self.c_struct,
                                self.pattern, self.p_v, self.p_s, self.row_ptr, self.col_idx, self.capacity,
                                self.nnz, self.o, self.lse, dense_below_tokens, stream), "crisp_forward")
        return self.o

    def poll(self, stream=None):
        for ws, name in ((self.route_ws, "route"), (self.select_ws, "select"), (self.prefill_ws, "prefill")):
            B.check(B.crisp_poll_device_status(ws, stream), f"device status ({name})")
