"""ctypes binding of libcrisp.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/crisp.h) and does nothing
but turn torch tensors into device pointers.  All arithmetic of the path runs in the CUDA library;
if the library cannot be loaded the import fails loudly: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcrisp.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_WORKSPACE = -3
ERR_CAPACITY = -4
ERR_CUDA = -5
ERR_DEVICE_TIMEOUT = -6
ERR_BAD_LIST = -7
PATTERN_PE, PATTERN_VS = 0, 1

EXPORTS = (
    "crisp_version", "crisp_status_string", "crisp_last_cuda_error", "crisp_workspace_bytes",
    "crisp_route", "crisp_route_static", "crisp_select", "crisp_sparse_prefill", "crisp_dense_prefill",
    "crisp_poll_device_status", "crisp_forward", "crisp_route_jsd", "crisp_varlen_layout",
    "crisp_forward_varlen", "crisp_selftest_bounded_wait", "crisp_profile_enable", "crisp_profile_read",
    "crisp_forward_host", "crisp_forward_host_stage_bytes",
)


class CrispParams(ctypes.Structure):
    """Mirror of `crisp_params` (include/crisp.h)."""
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("seq_len", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("block", ctypes.c_int32),
        ("sink_tokens", ctypes.c_int32), ("local_tokens", ctypes.c_int32),
        ("k_min_blocks", ctypes.c_int32), ("selector", ctypes.c_int32),
        ("force_pattern", ctypes.c_int32), ("tau", ctypes.c_float), ("alpha", ctypes.c_float),
        ("gamma", ctypes.c_float), ("softmax_scale", ctypes.c_float),
    ]


def make_params(seq_len: int, n_q_heads: int, n_kv_heads: int, *, sink_tokens: int = 128,
                local_tokens: int = 128, k_min_blocks: int = 8, selector: int = 0,
                force_pattern: int = 0, tau: float = 0.2, alpha: float = 1.0, gamma: float = 0.95,
                softmax_scale: float = 0.0, head_dim: int = 128, block: int = 128) -> CrispParams:
    return CrispParams(ctypes.sizeof(CrispParams), seq_len, n_q_heads, n_kv_heads, head_dim, block,
                       sink_tokens, local_tokens, k_min_blocks, selector, force_pattern, tau, alpha,
                       gamma, softmax_scale)


class CrispError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = f"{where}: {status_string(status)} ({status})"
        if status == ERR_CUDA:
            msg += f": {last_cuda_error()}"
        super().__init__(msg)


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """Load libcrisp.so (built in-tree by paper_2609_01925_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2609_01925_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    P = ctypes.POINTER(CrispParams)
    vp, sz, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64
    lib.crisp_version.restype = ctypes.c_int
    lib.crisp_version.argtypes = []
    lib.crisp_status_string.restype = ctypes.c_char_p
    lib.crisp_status_string.argtypes = [ctypes.c_int]
    lib.crisp_last_cuda_error.restype = ctypes.c_char_p
    lib.crisp_last_cuda_error.argtypes = []
    lib.crisp_workspace_bytes.restype = ctypes.c_int
    lib.crisp_workspace_bytes.argtypes = [P, ctypes.POINTER(sz), ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.crisp_route.restype = ctypes.c_int
    lib.crisp_route.argtypes = [P, vp, vp, vp, sz, vp, vp, vp, vp, vp]
    lib.crisp_route_static.restype = ctypes.c_int
    lib.crisp_route_static.argtypes = [P, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.crisp_select.restype = ctypes.c_int
    lib.crisp_select.argtypes = [P, vp, vp, vp, vp, vp, vp, sz, vp, vp, i64, vp, vp]
    lib.crisp_sparse_prefill.restype = ctypes.c_int
    lib.crisp_sparse_prefill.argtypes = [P, vp, vp, vp, vp, vp, vp, sz, vp, vp, vp]
    lib.crisp_dense_prefill.restype = ctypes.c_int
    lib.crisp_dense_prefill.argtypes = [P, vp, vp, vp, vp, sz, vp, vp, vp]
    lib.crisp_route_jsd.restype = ctypes.c_int
    lib.crisp_route_jsd.argtypes = [P, vp, vp, vp, vp, sz, ctypes.c_float, vp, vp, vp]
    lib.crisp_forward.restype = ctypes.c_int
    lib.crisp_forward.argtypes = [P, vp, vp, vp, vp, sz, vp, sz, vp, sz, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp,
                                  ctypes.c_int32, vp]
    lib.crisp_varlen_layout.restype = ctypes.c_int
    lib.crisp_varlen_layout.argtypes = [P, vp, ctypes.c_int32, i64, ctypes.c_int32, vp, vp]
    lib.crisp_forward_varlen.restype = ctypes.c_int
    lib.crisp_forward_varlen.argtypes = [P, vp, ctypes.c_int32, vp, vp, vp, vp, sz, vp, sz, vp, sz, vp, vp, vp, vp,
                                         vp, vp, i64, vp, vp, vp, vp, ctypes.c_int32, vp]
    lib.crisp_forward_host_stage_bytes.restype = sz
    lib.crisp_forward_host_stage_bytes.argtypes = [P, ctypes.c_int32]
    lib.crisp_forward_host.restype = ctypes.c_int
    lib.crisp_forward_host.argtypes = [P, vp, vp, vp, vp, ctypes.c_int32, vp, sz, vp, vp, vp]
    lib.crisp_profile_enable.restype = ctypes.c_int
    lib.crisp_profile_enable.argtypes = [ctypes.c_int]
    lib.crisp_profile_read.restype = ctypes.c_int
    lib.crisp_profile_read.argtypes = [ctypes.c_char_p, sz, ctypes.POINTER(ctypes.c_float), ctypes.c_int32,
                                       ctypes.POINTER(ctypes.c_int32)]
    lib.crisp_selftest_bounded_wait.restype = ctypes.c_int
    lib.crisp_selftest_bounded_wait.argtypes = [vp, sz, i64, vp]
    lib.crisp_poll_device_status.restype = ctypes.c_int
    lib.crisp_poll_device_status.argtypes = [vp, vp]
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def crisp_version() -> int:
    return load().crisp_version()


def status_string(status: int) -> str:
    return load().crisp_status_string(status).decode()


def last_cuda_error() -> str:
    return load().crisp_last_cuda_error().decode()


def crisp_workspace_bytes(p: CrispParams) -> Tuple[int, int, int]:
    a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    rc = load().crisp_workspace_bytes(ctypes.byref(p), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != OK:
        raise CrispError(rc, "crisp_workspace_bytes")
    return a.value, b.value, c.value


def crisp_route(p, q, k, ws, c_struct, pattern, p_v, p_s, stream=None) -> int:
    return load().crisp_route(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(ws), ws.numel() * ws.element_size(),
                              _ptr(c_struct), _ptr(pattern), _ptr(p_v), _ptr(p_s), _stream(stream))


ROUTE_STATIC_SCRATCH_BYTES = 4 << 20


def crisp_route_static(p, q, k, c_struct, pattern, p_v, p_s, device_status=None, stream=None) -> int:
    """crisp_route without a workspace argument: the scratch is a fixed 4 MiB array inside the library.

    For callers that cannot allocate device memory (see include/crisp.h).  Calls on one GPU must not
    overlap in time; problems whose route workspace exceeds ROUTE_STATIC_SCRATCH_BYTES are refused.
    """
    return load().crisp_route_static(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(c_struct), _ptr(pattern),
                                     _ptr(p_v), _ptr(p_s), _ptr(device_status), _stream(stream))


def crisp_select(p, q, k, pattern, p_v, p_s, ws, row_ptr, col_idx, capacity, nnz_needed, stream=None) -> int:
    return load().crisp_select(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(pattern), _ptr(p_v), _ptr(p_s),
                               _ptr(ws), ws.numel() * ws.element_size(), _ptr(row_ptr), _ptr(col_idx),
                               int(capacity), _ptr(nnz_needed), _stream(stream))


def crisp_sparse_prefill(p, q, k, v, row_ptr, col_idx, ws, o, lse=None, stream=None) -> int:
    return load().crisp_sparse_prefill(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(row_ptr),
                                       _ptr(col_idx), _ptr(ws), ws.numel() * ws.element_size(), _ptr(o),
                                       _ptr(lse), _stream(stream))


def crisp_dense_prefill(p, q, k, v, ws, o, lse=None, stream=None) -> int:
    return load().crisp_dense_prefill(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(ws),
                                      ws.numel() * ws.element_size(), _ptr(o), _ptr(lse), _stream(stream))


def crisp_route_jsd(p, q, k, p_v, select_ws, tau_jsd, jsd, pattern, stream=None) -> int:
    return load().crisp_route_jsd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(p_v), _ptr(select_ws),
                                  select_ws.numel() * select_ws.element_size(), float(tau_jsd), _ptr(jsd),
                                  _ptr(pattern), _stream(stream))


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def crisp_forward(p, q, k, v, route_ws, select_ws, prefill_ws, c_struct, pattern, p_v, p_s, row_ptr, col_idx,
                  capacity, nnz_needed, o, lse=None, dense_below_tokens=0, stream=None) -> int:
    return load().crisp_forward(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(route_ws), _nbytes(route_ws),
                                _ptr(select_ws), _nbytes(select_ws), _ptr(prefill_ws), _nbytes(prefill_ws),
                                _ptr(c_struct), _ptr(pattern), _ptr(p_v), _ptr(p_s), _ptr(row_ptr),
                                _ptr(col_idx), int(capacity), _ptr(nnz_needed), _ptr(o), _ptr(lse),
                                int(dense_below_tokens), _stream(stream))


def crisp_forward_host_stage_bytes(p, kv_groups_per_chunk: int) -> int:
    return int(load().crisp_forward_host_stage_bytes(ctypes.byref(p), int(kv_groups_per_chunk)))


def crisp_forward_host(p, q_host, k_host, v_host, o_host, kv_groups_per_chunk, stage, pattern_host=None,
                       stream=None):
    """Algorithm 1 on HOST tensors (CPU, ideally pinned), chunk by chunk of whole KV groups, copies overlapped with
    the kernels (see include/crisp.h).  `stage` is a device byte tensor of crisp_forward_host_stage_bytes bytes.
    Returns (status, blocks listed)."""
    for t in (q_host, k_host, v_host, o_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("crisp_forward_host takes contiguous CPU tensors")
    nnz = ctypes.c_int64(0)
    rc = load().crisp_forward_host(ctypes.byref(p), _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(o_host),
                                   int(kv_groups_per_chunk), _ptr(stage), _nbytes(stage), _ptr(pattern_host),
                                   ctypes.addressof(nnz), _stream(stream))
    return rc, int(nnz.value)


def _host_i64(values):
    arr = (ctypes.c_int64 * len(values))(*[int(x) for x in values])
    return arr


def crisp_varlen_layout(p, cu_seqlens, capacity, dense_below_tokens=0):
    """(blk_off, col_off) of a packed batch: where each sequence's outputs live (see include/crisp.h)."""
    batch = len(cu_seqlens) - 1
    cu = _host_i64(cu_seqlens)
    blk, col = (ctypes.c_int64 * (batch + 1))(), (ctypes.c_int64 * (batch + 1))()
    rc = load().crisp_varlen_layout(ctypes.byref(p), cu, batch, int(capacity), int(dense_below_tokens), blk, col)
    if rc != OK:
        raise CrispError(rc, "crisp_varlen_layout")
    return list(blk), list(col)


def crisp_forward_varlen(p, cu_seqlens, q, k, v, route_ws, select_ws, prefill_ws, c_struct, pattern, p_v, p_s,
                         row_ptr, col_idx, capacity, nnz_needed, device_status, o, lse=None, dense_below_tokens=0,
                         stream=None) -> int:
    """cu_seqlens: a host sequence of batch + 1 token offsets (list, tuple or CPU tensor)."""
    cu = _host_i64([int(x) for x in cu_seqlens])
    return load().crisp_forward_varlen(ctypes.byref(p), cu, len(cu) - 1, _ptr(q), _ptr(k), _ptr(v), _ptr(route_ws),
                                       _nbytes(route_ws), _ptr(select_ws), _nbytes(select_ws), _ptr(prefill_ws),
                                       _nbytes(prefill_ws), _ptr(c_struct), _ptr(pattern), _ptr(p_v), _ptr(p_s),
                                       _ptr(row_ptr), _ptr(col_idx), int(capacity), _ptr(nnz_needed),
                                       _ptr(device_status), _ptr(o), _ptr(lse), int(dense_below_tokens),
                                       _stream(stream))


def crisp_profile_enable(on: bool) -> int:
    return load().crisp_profile_enable(1 if on else 0)


def crisp_profile_read(max_records: int = 4096):
    """[(kernel name, milliseconds)] of the kernels launched since crisp_profile_enable(True), in launch order."""
    names = ctypes.create_string_buffer(64 * max_records)
    ms = (ctypes.c_float * max_records)()
    n = ctypes.c_int32(0)
    rc = load().crisp_profile_read(names, len(names), ms, max_records, ctypes.byref(n))
    if rc != OK:
        raise CrispError(rc, "crisp_profile_read")
    return list(zip(names.value.decode().split("\n")[:n.value], [float(x) for x in ms[:n.value]]))


def crisp_selftest_bounded_wait(ws, limit_ns, stream=None) -> int:
    return load().crisp_selftest_bounded_wait(_ptr(ws), _nbytes(ws), int(limit_ns), _stream(stream))


def crisp_poll_device_status(ws, stream=None) -> int:
    return load().crisp_poll_device_status(_ptr(ws), _stream(stream))


def check(rc: int, where: str) -> None:
    if rc != OK:
        raise CrispError(rc, where)
