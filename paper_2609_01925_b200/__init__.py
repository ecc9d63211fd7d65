"""B200 (sm_100a) implementation of CRISP's sparse-prefill attention path.

`binding` mirrors the C ABI of include/crisp.h one to one; `CrispLayer` is a small convenience
wrapper that owns the device buffers (torch is used for memory and streams only).
"""
from . import binding
from .binding import (CrispError, CrispParams, crisp_dense_prefill, crisp_poll_device_status, crisp_route,
                      crisp_select, crisp_sparse_prefill, crisp_version, crisp_workspace_bytes, make_params)
from .layer import CrispLayer

__all__ = ["binding", "CrispError", "CrispParams", "CrispLayer", "make_params", "crisp_version",
           "crisp_workspace_bytes", "crisp_route", "crisp_select", "crisp_sparse_prefill",
           "crisp_dense_prefill", "crisp_poll_device_status"]
