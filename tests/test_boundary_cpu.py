"""Host-side checks that need no GPU: the library loads, exports every declared symbol, validates
its arguments and sizes its workspaces.  No compute call is made."""
import ctypes
import os
import re

import pytest

import paper_2609_01925_b200 as crisp
from paper_2609_01925_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = B.load()
    header = open(os.path.join(ROOT, "include", "crisp.h")).read()
    declared = set(re.findall(r"\b(crisp_[a-z_]+)\s*\(", header))
    declared -= {"crisp_params", "crisp_status"}
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings():
    assert crisp.crisp_version() >= 100
    assert B.status_string(B.OK) == "ok"
    for code in (B.ERR_INVALID_ARG, B.ERR_UNSUPPORTED, B.ERR_WORKSPACE, B.ERR_CAPACITY, B.ERR_CUDA,
                 B.ERR_DEVICE_TIMEOUT, B.ERR_BAD_LIST):
        assert B.status_string(code) not in ("ok", "unknown status")
    assert B.status_string(12345) == "unknown status"


def test_params_struct_matches_header():
    assert ctypes.sizeof(B.CrispParams) == 15 * 4
    header = open(os.path.join(ROOT, "include", "crisp.h")).read()
    body = header[header.index("typedef struct crisp_params"):header.index("} crisp_params;")]
    fields = re.findall(r"^\s*(?:int32_t|float)\s+(\w+);", body, flags=re.M)
    assert fields == [f[0] for f in B.CrispParams._fields_]


def test_workspace_sizes_grow_with_the_problem():
    small = B.crisp_workspace_bytes(crisp.make_params(4096, 4, 1))
    big = B.crisp_workspace_bytes(crisp.make_params(32768, 32, 8))
    assert all(s > 0 for s in small) and all(b > s for s, b in zip(small, big))
    # 512k: everything must fit comfortably in 180 GB
    huge = B.crisp_workspace_bytes(crisp.make_params(524288, 32, 8))
    assert sum(huge) < 8 << 30


@pytest.mark.parametrize("kw,code", [
    (dict(seq_len=8192 * 128 + 1), B.ERR_UNSUPPORTED),   # more than 8192 blocks
    (dict(seq_len=0), B.ERR_INVALID_ARG),
    (dict(head_dim=64), B.ERR_UNSUPPORTED),
    (dict(block=64), B.ERR_UNSUPPORTED),
    (dict(n_q_heads=6, n_kv_heads=4), B.ERR_INVALID_ARG),
    (dict(n_q_heads=34, n_kv_heads=2), B.ERR_UNSUPPORTED),   # group of 17
    (dict(sink_tokens=0), B.ERR_INVALID_ARG),
    (dict(local_tokens=10 ** 7), B.ERR_INVALID_ARG),
    (dict(k_min_blocks=-1), B.ERR_INVALID_ARG),
    (dict(selector=3), B.ERR_INVALID_ARG),
    (dict(force_pattern=3), B.ERR_INVALID_ARG),
    (dict(alpha=-1.0), B.ERR_INVALID_ARG),
    (dict(gamma=0.0), B.ERR_INVALID_ARG),
    (dict(tau=float("nan")), B.ERR_INVALID_ARG),
    (dict(softmax_scale=-0.5), B.ERR_INVALID_ARG),
])
def test_invalid_parameters_are_rejected(kw, code):
    base = dict(seq_len=4096, n_q_heads=4, n_kv_heads=1)
    base.update(kw)
    n, hq, hkv = base.pop("seq_len"), base.pop("n_q_heads"), base.pop("n_kv_heads")
    p = crisp.make_params(n, hq, hkv, **base)
    with pytest.raises(crisp.CrispError) as e:
        B.crisp_workspace_bytes(p)
    assert e.value.status == code


@pytest.mark.parametrize("n", [1, 100, 128, 255])
def test_lengths_below_two_blocks_are_dense_only(n):
    """Routing needs two blocks (the noise floor divides by N_b - 2 and the proxy block needs a predecessor);
    dense attention does not: the workspace query says so, and the routed entry points refuse the length
    before they look at any pointer."""
    import ctypes
    p = crisp.make_params(n, 4, 1, sink_tokens=4, local_tokens=128)
    route_ws, select_ws, prefill_ws = B.crisp_workspace_bytes(p)
    assert route_ws == 0 and select_ws == 0 and prefill_ws > 0
    lib = B.load()
    assert lib.crisp_route(ctypes.byref(p), None, None, None, 0, None, None, None, None, None) == B.ERR_UNSUPPORTED
    assert lib.crisp_select(ctypes.byref(p), None, None, None, None, None, None, 0, None, None, 0, None,
                            None) == B.ERR_UNSUPPORTED
    assert lib.crisp_sparse_prefill(ctypes.byref(p), None, None, None, None, None, None, 0, None, None,
                                    None) == B.ERR_UNSUPPORTED


def test_varlen_layout_rule():
    """blk_off counts blocks of every sequence; col_off splits the capacity in proportion to the causal block
    counts of the routed sequences (dense and empty ones get nothing), with floor rounding."""
    p = crisp.make_params(4096, 4, 2, sink_tokens=4)
    lens = [300, 0, 1000, 128, 70, 2112]
    cu = [0]
    for x in lens:
        cu.append(cu[-1] + x)
    nb = [(x + 127) // 128 for x in lens]
    causal = [b * (b + 1) // 2 if x >= 256 else 0 for x, b in zip(lens, nb)]
    capacity = 4 * sum(causal) + 3
    blk, col = B.crisp_varlen_layout(p, cu, capacity)
    assert blk == [sum(nb[:i]) for i in range(len(lens) + 1)]
    assert col == [capacity * sum(causal[:i]) // sum(causal) for i in range(len(lens) + 1)]
    assert col[-1] == capacity and all(b >= a for a, b in zip(col, col[1:]))
    # the gate moves short sequences to dense: they lose their share
    blk2, col2 = B.crisp_varlen_layout(p, cu, capacity, dense_below_tokens=512)
    causal2 = [c if x >= 512 else 0 for c, x in zip(causal, lens)]
    assert blk2 == blk and col2 == [capacity * sum(causal2[:i]) // sum(causal2) for i in range(len(lens) + 1)]
    # nothing routed: every share is empty
    assert B.crisp_varlen_layout(p, [0, 100, 200], 1000)[1] == [0, 0, 0]
    with pytest.raises(crisp.CrispError):
        B.crisp_varlen_layout(p, [0, 300, 200], 1000)      # decreasing offsets
    with pytest.raises(crisp.CrispError):
        B.crisp_varlen_layout(p, [5, 300], 1000)           # must start at 0


def test_ragged_lengths_are_accepted():
    for n in (256, 257, 4096 + 64, 8192 * 128 - 5):
        sizes = B.crisp_workspace_bytes(crisp.make_params(n, 4, 1))
        assert all(s > 0 for s in sizes)


def test_abi_guard_and_null_pointers():
    lib = B.load()
    p = crisp.make_params(4096, 4, 1)
    p.struct_size = 8
    assert lib.crisp_workspace_bytes(ctypes.byref(p), None, None, None) == B.ERR_INVALID_ARG
    assert lib.crisp_workspace_bytes(None, None, None, None) == B.ERR_INVALID_ARG
    p = crisp.make_params(4096, 4, 1)
    assert lib.crisp_workspace_bytes(ctypes.byref(p), None, None, None) == B.OK
    # null data pointers are caught before anything is launched (no GPU needed)
    assert lib.crisp_route(ctypes.byref(p), None, None, None, 0, None, None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.crisp_select(ctypes.byref(p), None, None, None, None, None, None, 0, None, None, 0, None,
                            None) == B.ERR_INVALID_ARG
    assert lib.crisp_sparse_prefill(ctypes.byref(p), None, None, None, None, None, None, 0, None, None,
                                    None) == B.ERR_INVALID_ARG
    assert lib.crisp_dense_prefill(ctypes.byref(p), None, None, None, None, 0, None, None, None) == B.ERR_INVALID_ARG
    assert lib.crisp_poll_device_status(None, None) == B.ERR_INVALID_ARG


def test_misaligned_and_short_workspace_are_rejected():
    lib = B.load()
    p = crisp.make_params(4096, 4, 1)
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1004)
    assert lib.crisp_route(ctypes.byref(p), fake, fake, fake, 16, fake, fake, fake, fake, None) == B.ERR_WORKSPACE
    assert lib.crisp_route(ctypes.byref(p), fake, fake, odd, 1 << 30, fake, fake, fake, fake, None) == B.ERR_WORKSPACE
    assert lib.crisp_route(ctypes.byref(p), odd, fake, fake, 1 << 30, fake, fake, fake, fake, None) == B.ERR_INVALID_ARG
    assert lib.crisp_dense_prefill(ctypes.byref(p), fake, fake, fake, fake, 8, fake, None, None) == B.ERR_WORKSPACE
    assert lib.crisp_select(ctypes.byref(p), fake, fake, fake, fake, fake, fake, 1 << 30, fake, None, 5, fake,
                            None) == B.ERR_INVALID_ARG   # capacity > 0 without col_idx


def test_layer_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        crisp.CrispLayer(crisp.make_params(4096, 4, 1))


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_01925_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("no cpu or pytorch fallback", ""), f
