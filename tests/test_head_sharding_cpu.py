"""Head-sharded multi-GPU layout on CPU: two gloo ranks split the KV groups of one layer, every head is owned by
exactly one rank, a rank's input slice equals the corresponding slice of the full tensors, and what a rank would
compute for its heads (the oracle stands in for the kernels here) equals the single-rank result for those heads.
The GPU twin of this test runs both shards one after the other on one device (tests/test_gpu_head_sharding.py)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from workloads import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _workload():
    return synth.llama_shaped("shard-test", 1024, 8).with_(n_q_heads=8, n_kv_heads=4,
                                                            head_classes=("conc", "diffuse") * 4, k_min_blocks=2)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import crisp_oracle as orc
    from paper_2609_01925_b200 import sharding
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = _workload()
    groups = sharding.kv_groups_of_rank(w.n_kv_heads, rank, world)
    heads = sharding.q_heads_of_groups(groups, w.group)
    q, k, v = synth.make_qkv_kv_groups(w, groups)
    kw = dict(block=128, sink_tokens=w.sink_tokens, local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha,
              gamma=w.gamma, k_min_blocks=w.k_min_blocks)
    res = orc.layer_pipeline(q.float().numpy(), k.float().numpy(), **kw)      # local head j reads local KV head j // G
    lists = [[c.tolist() for c in r["cols"]] for r in res]
    ms = bench.max_over_ranks(10.0 + rank, dist, torch.device("cpu"))
    gathered = [None] * world
    dist.all_gather_object(gathered, heads)
    dist.barrier()
    out[rank] = dict(heads=heads, all_heads=gathered, q=q.float().numpy(), k=k.float().numpy(), lists=lists,
                     labels=[r["pattern"] for r in res], ms=ms, job=bench.job_ms_per_layer(ms, world, "kv-groups"))
    dist.destroy_process_group()


def test_two_ranks_partition_the_heads_and_reproduce_the_single_rank_results():
    from oracle import crisp_oracle as orc
    world = 2
    port = 29600 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    w = _workload()
    owned = sorted(h for r in range(world) for h in res[r]["heads"])
    assert owned == list(range(w.n_q_heads))                       # every head once
    assert res[0]["all_heads"] == [res[0]["heads"], res[1]["heads"]]
    assert res[0]["ms"] == res[1]["ms"] == 11.0 and res[0]["job"] == 11.0   # the layer takes as long as the slowest rank
    q, k, v = synth.make_qkv(w)
    kw = dict(block=128, sink_tokens=w.sink_tokens, local_tokens=w.local_tokens, tau=w.tau, alpha=w.alpha,
              gamma=w.gamma, k_min_blocks=w.k_min_blocks)
    full = orc.layer_pipeline(q.float().numpy(), k.float().numpy(), **kw)
    for r in range(world):
        heads = res[r]["heads"]
        kv_heads = sorted({h // w.group for h in heads})
        assert np.array_equal(res[r]["q"], q[:, heads].float().numpy())
        assert np.array_equal(res[r]["k"], k[:, kv_heads].float().numpy())
        for j, h in enumerate(heads):
            assert res[r]["labels"][j] == full[h]["pattern"]
            assert res[r]["lists"][j] == [c.tolist() for c in full[h]["cols"]]


def test_partition_rules():
    from paper_2609_01925_b200 import sharding
    import pytest
    assert sharding.kv_groups_of_rank(8, 3, 8) == [3]
    assert sharding.kv_groups_of_rank(8, 1, 3) == [1, 4, 7]
    assert sharding.q_heads_of_groups([1, 4], 4) == [4, 5, 6, 7, 16, 17, 18, 19]
    for world in (1, 2, 3, 4, 8):
        got = sorted(g for r in range(world) for g in sharding.kv_groups_of_rank(8, r, world))
        assert got == list(range(8))
    with pytest.raises(ValueError):
        sharding.kv_groups_of_rank(4, 0, 8)                        # more ranks than KV groups
    with pytest.raises(ValueError):
        sharding.kv_groups_of_rank(4, 4, 4)
