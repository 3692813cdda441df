"""The benchmark's multi-rank reduction (replicas: MAX of times, SUM of counts) under gloo, 2 ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t, n = bench.reduce_over_ranks([10.0 + rank, 3.0 - rank], [100 * (rank + 1), 7], dist)
    out.put((rank, t, n))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, n in res:
        assert t == [11.0, 3.0]          # slowest rank decides the time
        assert n == [300.0, 14.0]        # tokens and launches add up over the replicas


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([5.0], [3]) == ([5.0], [3.0])
    # whole-job tokens/s of N replicas = sum of tokens / slowest time
    t, n = [12.0], [96.0 * 2]
    assert n[0] / (t[0] * 1e-3) == 16000.0


def test_workload_capacity_and_bytes():
    sys.path.insert(0, ROOT)
    import bench
    cfg = bench.workload(100)
    assert cfg.S_max >= 512 + 100 * 5 + cfg.N and cfg.S_max % 128 == 0
    ab = bench.algorithmic_bytes_per_step(cfg, 512.0)
    assert ab["verify_weights"] == 32 * 202375168 * 2 + 32000 * 4096 * 2     # 7B layer matrices + LM head
    assert ab["draft_weights"] == 8 * 4096 * 4096 * 2 + 32000 * 4096 * 2
    assert ab["kv"] == 32 * 512 * 32 * 128 * 2 * 2
