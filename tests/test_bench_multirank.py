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
    """Capacity rule and the algorithmic bytes / flops of a step, against numbers worked out by hand."""
    sys.path.insert(0, ROOT)
    import bench
    from workloads import T13_EAGLE, T7_EAGLE, T7_MEDUSA
    cfg = bench.with_capacity(T7_MEDUSA, 100)
    assert cfg.S_max >= 512 + 100 * 5 + cfg.N and cfg.S_max % 128 == 0
    ab = bench.algorithmic_work(cfg, 512.0)
    layer7 = 202375168 * 2                                                    # 7B layer matrices, bf16
    assert ab["verify_weights"] == 32 * layer7 + 32000 * 4096 * 2            # + LM head
    assert ab["draft_weights"] == 8 * 4096 * 4096 * 2 + 32000 * 4096 * 2
    assert ab["kv"] == 32 * 512 * 32 * 128 * 2 * 2
    # EAGLE-style head, K = 2, 5 passes: fc + 2 layers + LM head per pass; the head's own cache per layer and pass
    ab = bench.algorithmic_work(T7_EAGLE, 1024.0)
    assert ab["draft_weights"] == 5 * (2 * 4096 * 4096 * 2 + 2 * layer7 + 32000 * 4096 * 2)
    assert ab["kv"] == (32 + 5 * 2) * 1024 * 4096 * 2 * 2
    # flops: 2 per weight and row; verify rows = B x N, draft rows = B x (1 + 4 x 10)
    ab = bench.algorithmic_work(T13_EAGLE, 1280.0)
    layer13 = (4 * 5120 * 5120 + 3 * 5120 * 13824) * 2
    vw = 40 * layer13 + 32000 * 5120 * 2
    pw = 2 * 5120 * 5120 * 2 + 2 * layer13 + 32000 * 5120 * 2
    assert ab["verify_weights"] == vw
    assert ab["flops"] == 2.0 * (vw / 2) * 256 + 2.0 * (pw / 2) * 4 * 41
    peaks = {"hbm_gbs": 6400.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "test"}
    sr = bench.step_roofline(T13_EAGLE, 1280.0, 20.0, peaks)
    assert sr["bound"] in ("hbm", "tensor") and 0 < sr["frac_of_peak"] < 1
    assert abs(sr["frac_of_peak"] - max(sr["ideal_ms_hbm"], sr["ideal_ms_tensor"]) / 20.0) < 1e-12
