"""Seeded synthetic Q/K/V with planted sink, vertical, slash and diffuse structure.

This module only *makes inputs*.  It holds none of the method's arithmetic (no
softmax, no block scores, no selection): the CPU oracle and the CUDA path both
receive the tensors built here and nothing else is shared between them.

Recipe (one attention layer, head_dim d = 128, rotary pairs p = 0..63 on dims
(p, p + 64), angle pos * theta**(-p/64)):

* three orthogonal sub-spaces make the logits decompose as
  noise(i, j) + vertical(j) + slash(i - j):
    U = rotary pairs 52..63 (24 dims), written AFTER the rotation, so it does
        not depend on position;
    W = rotary pairs 0..31 (64 dims), written BEFORE the rotation, so the dot
        product depends on i - j only;
    noise = pairs 32..51 (40 dims), iid normal.
* keys (one set per KV head): noise ~ N(0, 1); K[j] += s_j on U with s_j the
  sink scale for j < 4, the column scale for planted columns and 0 otherwise;
  before the rotation K0[j] += c_sl * sum_m a_m R(delta_m) 1_W, which plants
  one slash line per offset delta_m.
* query heads by class: "conc" (noise N(0,1), + 1_W before and + 1_U after the
  rotation), "sink" (+ 1_U only), "slash" (+ 1_W only), "diffuse" (noise
  N(0, 0.25), nothing planted).
* V ~ N(0, 1).  Everything is rounded to bf16 once.

Random numbers come from a counter-based generator (a splitmix64-style hash of
(seed, stream, element index) followed by Box-Muller), written with integer
torch ops so that any chunk can be produced on any device independently.
Transcendentals differ in the last bit between CPU and CUDA, so a tensor is
built once, on one device, and copied to whoever needs it.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Tuple

import torch

HEAD_DIM = 128
BLOCK = 128
N_PAIRS = 64
U_PAIRS = (52, 64)   # [lo, hi) rotary pairs of the vertical sub-space
W_PAIRS = (0, 32)    # rotary pairs of the slash sub-space
NOISE_PAIRS = (32, 52)

_M64 = (1 << 64)


def _s64(x: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    x &= _M64 - 1
    return x - _M64 if x >= (1 << 63) else x


_C1 = _s64(0x9E3779B97F4A7C15)
_C2 = _s64(0xBF58476D1CE4E5B9)
_C3 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """splitmix64-style mix of (seed, stream, idx); int64 in, int64 out (wrapping)."""
    base = _s64(seed * 0x9E3779B97F4A7C15 + (stream + 1) * 0xD1B54A32D192ED03)
    z = idx + base
    z = (z ^ _lsr(z, 30)) * _C2
    z = (z ^ _lsr(z, 27)) * _C3
    z = z ^ _lsr(z, 31)
    # second round decorrelates neighbouring counters of different streams
    z = (z + _C1)
    z = (z ^ _lsr(z, 30)) * _C2
    z = (z ^ _lsr(z, 27)) * _C3
    return z ^ _lsr(z, 31)


def normal(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """One standard normal (fp32) per int64 counter in ``idx``."""
    z = hash64(seed, stream, idx)
    a = _lsr(z, 40)                      # top 24 bits
    b = _lsr(z, 16) & 0xFFFFFF           # next 24 bits
    u1 = (a.to(torch.float32) + 1.0) * (1.0 / 16777216.0)     # (0, 1]
    u2 = b.to(torch.float32) * (1.0 / 16777216.0)             # [0, 1)
    r = torch.sqrt(-2.0 * torch.log(u1))
    return r * torch.cos((2.0 * math.pi) * u2)


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape, planted structure and method parameters of one synthetic layer."""
    name: str
    seq_len: int
    n_q_heads: int
    n_kv_heads: int
    rope_theta: float
    head_classes: Tuple[str, ...]           # per query head
    sink_scale: float = 8.0
    n_sink_tokens: int = 4                   # planted sink tokens 0..3
    n_columns: int = 0
    column_scale: float = 4.0
    slash_offsets: Tuple[int, ...] = ()
    slash_amps: Tuple[float, ...] = ()
    c_sl: float = 1.5
    seed: int = 0
    # method parameters the config is run with
    alpha: float = 1.0
    tau: float = 0.2
    gamma: float = 0.95
    k_min_blocks: int = 8
    sink_tokens: int = 4                     # w_sink used by the router
    local_tokens: int = 128                  # w_local used by the router

    @property
    def n_blocks(self) -> int:
        return -(-self.seq_len // BLOCK)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _alternating(n_heads: int) -> Tuple[str, ...]:
    return tuple("conc" if h % 2 == 0 else "diffuse" for h in range(n_heads))


def _offsets_for(n: int) -> Tuple[Tuple[int, ...], Tuple[float, ...]]:
    offs = tuple(o for o in (1, 96, 1056, 20000) if o < n - BLOCK)
    return offs, tuple(1.0 for _ in offs)


def llama_shaped(name: str, n: int, n_columns: int, seed: int = 0, **kw) -> Workload:
    offs, amps = _offsets_for(n)
    return Workload(name=name, seq_len=n, n_q_heads=32, n_kv_heads=8, rope_theta=5e5,
                    head_classes=_alternating(32), n_columns=n_columns,
                    slash_offsets=offs, slash_amps=amps, seed=seed, **kw)


def qwen_shaped(name: str, n: int, seed: int = 0, **kw) -> Workload:
    offs, _ = _offsets_for(n)
    amps = tuple(1.5 if o == 1 else 1.0 for o in offs)
    classes = tuple(("sink", "slash", "diffuse", "diffuse")[h % 4] for h in range(28))
    return Workload(name=name, seq_len=n, n_q_heads=28, n_kv_heads=4, rope_theta=1e6,
                    head_classes=classes, sink_scale=16.0, n_columns=0,
                    slash_offsets=offs, slash_amps=amps, seed=seed, **kw)


def tiny(seed: int = 0, n: int = 4096) -> Workload:
    return Workload(name="Tiny", seq_len=n, n_q_heads=4, n_kv_heads=1, rope_theta=5e5,
                    head_classes=("conc", "conc", "diffuse", "diffuse"), n_columns=16,
                    seed=seed, tau=0.1)


CONFIGS: Dict[str, Workload] = {
    "Tiny": tiny(),
    "L32k": llama_shaped("L32k", 32768, 64),
    "L128k": llama_shaped("L128k", 131072, 64),
    "Q256k": qwen_shaped("Q256k", 262144),
    "L512k": llama_shaped("L512k", 524288, 256),
}

# streams of the counter-based generator
_ST_KNOISE, _ST_QNOISE, _ST_V, _ST_COLS = 0, 1, 2, 3


def planted_columns(w: Workload, kv_head: int) -> List[int]:
    """Token positions of the planted vertical columns of one KV head (in [B, n-B))."""
    if w.n_columns == 0 or w.seq_len <= 2 * BLOCK:
        return []
    idx = torch.arange(w.n_columns, dtype=torch.int64) + kv_head * 1_000_003
    z = hash64(w.seed, _ST_COLS, idx)
    span = w.seq_len - 2 * BLOCK
    cols = (_lsr(z, 11) % span) + BLOCK
    return [int(c) for c in cols.tolist()]


def _inv_freq(w: Workload, device) -> torch.Tensor:
    p = torch.arange(N_PAIRS, dtype=torch.float64, device=device)
    return torch.exp(-(p / N_PAIRS) * math.log(w.rope_theta))


def _rotate(x: torch.Tensor, ang: torch.Tensor) -> torch.Tensor:
    """Rotary embedding: x [T, H, 128] fp32, ang [T, 64] fp64 (pairs (p, p+64))."""
    c = torch.cos(ang).to(torch.float32)[:, None, :]
    s = torch.sin(ang).to(torch.float32)[:, None, :]
    x1, x2 = x[..., :N_PAIRS], x[..., N_PAIRS:]
    return torch.cat((x1 * c - x2 * s, x1 * s + x2 * c), dim=-1)


def _pair_mask(lo_hi: Tuple[int, int], device) -> torch.Tensor:
    m = torch.zeros(HEAD_DIM, dtype=torch.float32, device=device)
    lo, hi = lo_hi
    m[lo:hi] = 1.0
    m[N_PAIRS + lo:N_PAIRS + hi] = 1.0
    return m


def _chunk_counters(t0: int, t1: int, n_heads: int, device) -> torch.Tensor:
    """Element counters ((token * H + head) * 128 + dim) of tokens [t0, t1)."""
    t = torch.arange(t0, t1, dtype=torch.int64, device=device)[:, None, None]
    h = torch.arange(n_heads, dtype=torch.int64, device=device)[None, :, None]
    c = torch.arange(HEAD_DIM, dtype=torch.int64, device=device)[None, None, :]
    return (t * n_heads + h) * HEAD_DIM + c


def make_k_chunk(w: Workload, t0: int, t1: int, device="cpu") -> torch.Tensor:
    """Keys of tokens [t0, t1): [t1-t0, H_kv, 128] bf16."""
    dev = torch.device(device)
    H = w.n_kv_heads
    noise_m = _pair_mask(NOISE_PAIRS, dev)
    u_m = _pair_mask(U_PAIRS, dev)
    x = normal(w.seed, _ST_KNOISE, _chunk_counters(t0, t1, H, dev)) * noise_m
    pos = torch.arange(t0, t1, dtype=torch.float64, device=dev)
    inv = _inv_freq(w, dev)
    x = _rotate(x, pos[:, None] * inv[None, :])
    # slash lines: c_sl * sum_m a_m R(j + delta_m) 1_W  (already rotated)
    if w.slash_offsets:
        lo, hi = W_PAIRS
        acc1 = torch.zeros(t1 - t0, hi - lo, dtype=torch.float64, device=dev)
        acc2 = torch.zeros_like(acc1)
        for delta, amp in zip(w.slash_offsets, w.slash_amps):
            ang = (pos[:, None] + float(delta)) * inv[None, lo:hi]
            cs, sn = torch.cos(ang), torch.sin(ang)
            acc1 += amp * (cs - sn)
            acc2 += amp * (sn + cs)
        x[:, :, lo:hi] += (w.c_sl * acc1).to(torch.float32)[:, None, :]
        x[:, :, N_PAIRS + lo:N_PAIRS + hi] += (w.c_sl * acc2).to(torch.float32)[:, None, :]
    # vertical structure on U (position independent)
    s = torch.zeros(t1 - t0, H, dtype=torch.float32, device=dev)
    n_sink_here = max(0, min(w.n_sink_tokens, t1) - t0)
    if n_sink_here > 0:
        s[:n_sink_here, :] = w.sink_scale
    for kv in range(H):
        for col in planted_columns(w, kv):
            if t0 <= col < t1:
                s[col - t0, kv] = w.column_scale
    x = x + s[:, :, None] * u_m
    return x.to(torch.bfloat16)


def make_q_chunk(w: Workload, t0: int, t1: int, device="cpu") -> torch.Tensor:
    """Queries of tokens [t0, t1): [t1-t0, H_q, 128] bf16."""
    dev = torch.device(device)
    H = w.n_q_heads
    noise_m = _pair_mask(NOISE_PAIRS, dev)
    u_m = _pair_mask(U_PAIRS, dev)
    w_m = _pair_mask(W_PAIRS, dev)
    std = torch.tensor([0.5 if c == "diffuse" else 1.0 for c in w.head_classes],
                       dtype=torch.float32, device=dev)
    has_w = torch.tensor([1.0 if c in ("conc", "slash") else 0.0 for c in w.head_classes],
                         dtype=torch.float32, device=dev)
    has_u = torch.tensor([1.0 if c in ("conc", "sink") else 0.0 for c in w.head_classes],
                         dtype=torch.float32, device=dev)
    x = normal(w.seed, _ST_QNOISE, _chunk_counters(t0, t1, H, dev)) * noise_m
    x = x * std[None, :, None] + has_w[None, :, None] * w_m
    pos = torch.arange(t0, t1, dtype=torch.float64, device=dev)
    x = _rotate(x, pos[:, None] * _inv_freq(w, dev)[None, :])
    x = x + has_u[None, :, None] * u_m
    return x.to(torch.bfloat16)


def make_v_chunk(w: Workload, t0: int, t1: int, device="cpu") -> torch.Tensor:
    dev = torch.device(device)
    x = normal(w.seed, _ST_V, _chunk_counters(t0, t1, w.n_kv_heads, dev))
    return x.to(torch.bfloat16)


def make_qkv(w: Workload, device="cpu", chunk_tokens: int = 8192):
    """Q [n, H_q, 128], K, V [n, H_kv, 128] in bf16 on ``device``, built chunk by chunk."""
    dev = torch.device(device)
    n = w.seq_len
    q = torch.empty(n, w.n_q_heads, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    k = torch.empty(n, w.n_kv_heads, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    v = torch.empty(n, w.n_kv_heads, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    for t0 in range(0, n, chunk_tokens):
        t1 = min(n, t0 + chunk_tokens)
        q[t0:t1] = make_q_chunk(w, t0, t1, dev)
        k[t0:t1] = make_k_chunk(w, t0, t1, dev)
        v[t0:t1] = make_v_chunk(w, t0, t1, dev)
    return q, k, v


def make_qkv_kv_groups(w: Workload, kv_groups, device="cpu", chunk_tokens: int = 8192):
    """The slice of make_qkv(w) that belongs to the given KV heads: K, V [n, len(kv_groups), 128] and the
    Q of their query heads [n, G * len(kv_groups), 128] (group-major, as a head-sharded rank stores them).
    Every element equals the corresponding element of the full tensors."""
    dev = torch.device(device)
    n, g = w.seq_len, w.group
    kv_idx = torch.tensor(list(kv_groups), dtype=torch.int64, device=dev)
    q_idx = (kv_idx[:, None] * g + torch.arange(g, dtype=torch.int64, device=dev)[None, :]).reshape(-1)
    q = torch.empty(n, q_idx.numel(), HEAD_DIM, dtype=torch.bfloat16, device=dev)
    k = torch.empty(n, kv_idx.numel(), HEAD_DIM, dtype=torch.bfloat16, device=dev)
    v = torch.empty(n, kv_idx.numel(), HEAD_DIM, dtype=torch.bfloat16, device=dev)
    for t0 in range(0, n, chunk_tokens):
        t1 = min(n, t0 + chunk_tokens)
        q[t0:t1] = make_q_chunk(w, t0, t1, dev)[:, q_idx]
        k[t0:t1] = make_k_chunk(w, t0, t1, dev)[:, kv_idx]
        v[t0:t1] = make_v_chunk(w, t0, t1, dev)[:, kv_idx]
    return q, k, v


def random_qkv(n: int, n_q_heads: int, n_kv_heads: int, seed: int, device="cpu",
               scale: float = 1.0):
    """Unstructured iid N(0, scale^2) inputs of an arbitrary shape (edge-case tests)."""
    w = Workload(name="iid", seq_len=n, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                 rope_theta=5e5, head_classes=("diffuse",) * n_q_heads, seed=seed)
    dev = torch.device(device)
    q = normal(seed, 11, _chunk_counters(0, n, n_q_heads, dev)) * scale
    k = normal(seed, 12, _chunk_counters(0, n, n_kv_heads, dev)) * scale
    v = normal(seed, 13, _chunk_counters(0, n, n_kv_heads, dev))
    del w
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
