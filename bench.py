#!/usr/bin/env python
"""Benchmark of the CRISP sparse-prefill hot path on B200.

One step = one pass of the whole hot path over one synthetic layer: crisp_route -> crisp_select ->
crisp_sparse_prefill (Algorithm 1).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload L512k] [--impl crisp|reference]

`value` is ms per layer of the whole path with inputs resident in HBM; `e2e` is the same through the
C ABI with HOST buffers (pinned host -> device copies of Q, K, V and a device -> host copy of O inside the
timed region).  The dense kernel (crisp_dense_prefill) is timed on the same inputs for the speedup.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import synth

FLOP_PER_BLOCK = 4 * 128 ** 3          # QK^T + PV of one 128 x 128 x 128 block pair
# kernels launched per step: route 5, select 16, sparse prefill 4 (merge, 2 x schedule, attention)
LAUNCHES_ROUTE, LAUNCHES_SELECT, LAUNCHES_PREFILL = 5, 16, 4


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"],
                    bf16_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(w, q, k, v, seed=0, blocks_per_head=4):
    """Times the fp64 oracle (as it stands) on a bounded sample of the workload and extrapolates to
    ms/layer: route+select of two heads (one per class) scaled to H_q, attention of a few query
    blocks scaled by the number of listed blocks.  Returns (ms_per_layer, description, cores)."""
    from oracle import crisp_oracle as orc
    hq, hkv, nb = w.n_q_heads, w.n_kv_heads, w.n_blocks
    classes = {}
    for h, c in enumerate(w.head_classes):
        classes.setdefault(c, h)
    heads = sorted(classes.values())[:2]
    kw = dict(block=128, sink_tokens=w.sink_tokens, local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha,
              gamma=w.gamma, k_min_blocks=w.k_min_blocks)
    t_sel, t_attn, blocks_done, nnz_est = 0.0, 0.0, 0, 0.0
    rng = np.random.default_rng(seed)
    for h in heads:
        qh = q[:, h].float().cpu().numpy()
        kh = k[:, h // w.group].float().cpu().numpy()
        vh = v[:, h // w.group].float().cpu().numpy()
        t0 = time.perf_counter()
        res = orc.head_pipeline(qh, kh, **kw)
        t_sel += time.perf_counter() - t0
        lens = np.array([len(c) for c in res["cols"]])
        nnz_est += lens.sum() * (sum(1 for c in w.head_classes if c == w.head_classes[h]))
        # a few query blocks, kept small enough for a bounded run
        order = np.argsort(lens)
        picks = [int(order[(2 * i + 1) * len(order) // (2 * blocks_per_head)]) for i in range(blocks_per_head)]
        for m in picks:
            t0 = time.perf_counter()
            orc.sparse_attention_block(qh, kh, vh, m, res["cols"][m], 128)
            t_attn += time.perf_counter() - t0
            blocks_done += len(res["cols"][m])
    per_head_sel = t_sel / len(heads)
    per_block = t_attn / max(blocks_done, 1)
    # heads of classes not sampled are counted like the nearest sampled class
    covered = sum(1 for c in w.head_classes if classes[c] in heads)
    nnz_est *= hq / max(covered, 1)
    ms = (per_head_sel * hq + per_block * nnz_est) * 1e3
    desc = (f"oracle route+select on heads {heads} (x{hq}/{len(heads)}), exact attention on "
            f"{blocks_done} listed blocks extrapolated to ~{int(nnz_est)} blocks")
    cores = torch.get_num_threads()
    return ms, desc, cores


def ncu_traffic_bytes(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` from the committed ncu summary of `workload`, or None."""
    path = os.path.join(ROOT, "profiles", f"dram_traffic_{workload}_ncu.md")
    if not os.path.exists(path):
        return None
    key = f"traffic_bytes_per_launch {kernel} {workload} ="
    with open(path) as f:
        for line in f:
            if line.startswith(key):
                return int(line.split("=")[1])
    return None


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's (all ranks run the same number of steps)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_ms_per_layer(ms_per_step: float, world: int) -> float:
    """Weak scaling: every rank processes one layer per step, so the job does `world` layers per step."""
    return ms_per_step / world


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="L512k", choices=list(synth.CONFIGS))
    ap.add_argument("--seq-len", type=int, default=0,
                    help="instead of a named workload: the Llama-shaped recipe (32/8 heads) at this many tokens "
                         "(context-length sweeps)")
    ap.add_argument("--impl", default="crisp", choices=["crisp", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = synth.CONFIGS[args.workload]
    if args.seq_len > 0:
        w = synth.llama_shaped(f"Llama-shaped-{args.seq_len}", args.seq_len, n_columns=max(16, args.seq_len // 2048))
    config = {"workload": f"{w.name}: n={w.seq_len}, H_q/H_kv={w.n_q_heads}/{w.n_kv_heads}, d=128, B=128, "
                          f"alpha={w.alpha}, tau={w.tau}, gamma={w.gamma}, w_sink={w.sink_tokens}, "
                          f"w_local={w.local_tokens}, k_min={w.k_min_blocks}",
              "layers_per_gpu": 1, "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
              "l2": "inputs larger than L2 (no flush)" if w.seq_len >= 131072 else "L2 flushed between steps"}

    if args.impl == "reference":
        if rank != 0:
            return
        dev = "cuda" if torch.cuda.is_available() else "cpu"
        q, k, v = synth.make_qkv(w, device=dev)
        times, desc, cores = [], "", 0
        for i in range(max(args.steps, 1)):
            ms, desc, cores = oracle_sample(w, q, k, v, seed=i)
            times.append(ms)
        val = statistics.median(times)
        print(json.dumps({
            "impl": "reference", "metric": "prefill attention ms/layer (route+select+sparse prefill)",
            "value": val, "unit": "ms/layer", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": val, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": "ms/layer", "cores": cores, "kind": "oracle",
                             "sample": desc + " (extrapolated)"},
            "e2e": {"value": val, "unit": "ms/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the product path has no CPU fallback)")
    import paper_2609_01925_b200 as crisp
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()

    q, k, v = synth.make_qkv(w.with_(seed=w.seed + rank), device=dev)
    p = crisp.make_params(w.seq_len, w.n_q_heads, w.n_kv_heads, sink_tokens=w.sink_tokens,
                          local_tokens=w.local_tokens, k_min_blocks=w.k_min_blocks, tau=w.tau, alpha=w.alpha,
                          gamma=w.gamma)
    layer = crisp.CrispLayer(p, device=dev)
    flush = None
    if w.seq_len < 131072:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    stage_ms = {"route": [], "select": [], "sparse_prefill": []}

    def step(record: bool):
        if flush is not None:
            flush.zero_()
        e = [ev() for _ in range(4)]
        e[0].record(); layer.route(q, k)
        e[1].record(); layer.select(q, k)
        e[2].record(); layer.sparse_prefill(q, k, v)
        e[3].record()
        return e if record else None

    for _ in range(args.warmup):
        step(False)
    layer.poll()
    nnz = int(layer.nnz.item())
    total_causal = w.n_q_heads * w.n_blocks * (w.n_blocks + 1) // 2

    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t_start, t_end = ev(), ev()
    t_start.record()
    recs = [step(True) for _ in range(args.steps)]
    t_end.record()
    barrier()
    total_ms = t_start.elapsed_time(t_end)
    for e in recs:
        stage_ms["route"].append(e[0].elapsed_time(e[1]))
        stage_ms["select"].append(e[1].elapsed_time(e[2]))
        stage_ms["sparse_prefill"].append(e[2].elapsed_time(e[3]))
    layer.poll()

    # dense baseline on the same inputs (own kernel), same protocol
    dense_ms = []
    for i in range(3 + min(args.steps, 3)):
        if flush is not None:
            flush.zero_()
        a, b = ev(), ev()
        a.record(); layer.dense_prefill(q, k, v); b.record()
        torch.cuda.synchronize()
        if i >= 3:
            dense_ms.append(a.elapsed_time(b))
    layer.poll()
    clocks = sampler.stop()

    # A step's time runs from its first launch to its last kernel's end (CUDA events on the launching stream).
    # Without an L2 flush the steps are back to back and this equals the bracket around all K steps; with a
    # flush (small workloads) it leaves the flush kernel between two steps out of the path's time.
    step_ms = [e[0].elapsed_time(e[3]) for e in recs]
    per_step = total_ms / args.steps if flush is None else sum(step_ms) / len(step_ms)
    ms_per_step = max_over_ranks(per_step, dist, dev)
    med = {kk: statistics.median(vv) for kk, vv in stage_ms.items()}
    dense = statistics.median(dense_ms)
    sparse_tflops = nnz * FLOP_PER_BLOCK / (med["sparse_prefill"] * 1e-3) / 1e12
    dense_tflops = total_causal * FLOP_PER_BLOCK / (dense * 1e-3) / 1e12
    peak = peaks["bf16_sustained"] if med["sparse_prefill"] > 50.0 else peaks["bf16_burst"]

    # end to end through the C ABI with host buffers
    e2e = None
    if not args.no_e2e:
        qh = q.cpu().pin_memory(); kh = k.cpu().pin_memory(); vh = v.cpu().pin_memory()
        oh = torch.empty(layer.o.shape, dtype=layer.o.dtype).pin_memory()
        qd, kd, vd = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        e2e_steps = min(args.steps, 3)
        for i in range(1 + e2e_steps):
            if i == 1:
                barrier()
                a = ev(); a.record()
            qd.copy_(qh, non_blocking=True); kd.copy_(kh, non_blocking=True); vd.copy_(vh, non_blocking=True)
            layer.forward(qd, kd, vd)
            oh.copy_(layer.o, non_blocking=True)
        b = ev(); b.record()
        barrier()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / e2e_steps, dist, dev)
        h2d = sum(x.numel() * x.element_size() for x in (qh, kh, vh))
        d2h = oh.numel() * oh.element_size()
        e2e = {"value": job_ms_per_layer(e2e_ms, world), "unit": "ms/layer", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        del qh, kh, vh, oh, qd, kd, vd

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ms, desc, cores = oracle_sample(w, q, k, v)
        cpu_baseline = {"value": ms, "unit": "ms/layer", "cores": cores, "kind": "oracle",
                        "sample": desc + " (extrapolated)"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    out = {
        "metric": "prefill attention ms/layer (route+select+sparse prefill)",
        "value": job_ms_per_layer(ms_per_step, world), "unit": "ms/layer", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
        "stages_ms": med, "dense_prefill_ms": dense, "speedup_vs_own_dense": dense / ms_per_step,
        "blocks_computed": nnz, "blocks_causal": total_causal, "block_fraction": nnz / total_causal,
        "sparse_tflops_on_computed_blocks": sparse_tflops, "dense_tflops": dense_tflops,
        "tc_frac_sparse_of_measured_sustained": sparse_tflops / peaks["bf16_sustained"],
        "tc_frac_dense_of_measured_sustained": dense_tflops / peaks["bf16_sustained"],
        "tc_frac_sparse_of_nominal_2250": sparse_tflops / 2250.0,
        "paper_context": "paper reports 5.17x-5.40x over FlashAttention at 512k on one H100 (real model heads)",
        "roofline": {"bound": "tensor", "kernel": "prefill_kernel<sparse>", "achieved": sparse_tflops,
                     "peak": peak, "unit": "TFLOP/s", "frac": sparse_tflops / peak,
                     "peak_source": f"{peaks['source']} ({'sustained' if peak == peaks['bf16_sustained'] else 'burst'})",
                     "traffic": ncu_traffic_bytes("prefill_kernel<sparse>", w.name),
                     "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum)",
                     "algorithmic_flop_per_launch": nnz * FLOP_PER_BLOCK},
        "cpu_baseline": cpu_baseline, "e2e": e2e,
        "gpu_launches": args.steps * (LAUNCHES_ROUTE + LAUNCHES_SELECT + LAUNCHES_PREFILL),
        "clocks": clocks,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
