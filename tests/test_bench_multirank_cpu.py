"""The N > 1 path of bench.py on CPU: two gloo ranks agree on the max-over-ranks step time and the
job-level metric (one independent layer per rank, no data-path collective)."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.job_ms_per_layer(ms, world))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_rank_and_scale_the_job_metric():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1] == (15.0, 7.5)


def test_single_rank_helpers_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, None, None) == 3.25
    assert bench.job_ms_per_layer(8.0, 1) == 8.0


def test_reference_arm_prints_one_json_line_on_cpu():
    """`--impl reference` times the CPU oracle on a bounded sample and needs no GPU."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                        "Tiny", "--steps", "1"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "ms/layer" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["higher_is_better"] is False
