#!/usr/bin/env python
"""Benchmark of the draft-then-verify step (speculative decoding with K-layer draft heads).

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A step is one whole iteration of the hot path (draft, tree expansion, verification of the whole
tree in one target forward, greedy acceptance + KV compaction) over one batch.  The workload is
the 7B-shaped target in bf16 with Medusa-style heads (4 heads x K=2 residual blocks, shared LM
head), a static 64-node tree and a 512-token context; weights are seeded N(0, 0.02) and the
prompt is seeded uniform token ids.  Random heads accept nothing, so the accepted length of each
step is forced from a seeded schedule (Poisson clipped to [1, 5], mean ~2.9 tokens per step).

Prints one JSON line.  With N > 1 every rank runs an independent replica (sequences share only
read-only weights, so there is no data-path collective) and the value is the whole job's.
`--impl reference` times the CPU oracle on the host cores instead (a deliberately slow baseline).
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

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import T7_MEDUSA  # noqa: E402
from workloads.generate import (WeightStore, forced_lengths, medusa_static_tree, prompts,  # noqa: E402
                                random_kv, normal_tensor, uniform_ints, weight_shapes)

METRIC = "spec_decode_tokens_per_s"
UNIT = "tokens/s"
FORCED_LAM, FORCED_LO, FORCED_HI = 3.0, 1, 5


def workload(steps_total: int):
    # capacity for the context, every step's growth and one tree
    s_max = 512 + steps_total * FORCED_HI + T7_MEDUSA.N + 64
    s_max = (s_max + 127) // 128 * 128
    return T7_MEDUSA.with_(S_max=max(s_max, 1024))


def workload_desc(cfg):
    return {"workload": cfg.name, "target": "7B-shaped Llama (32 layers, hidden 4096, 32x128 heads, FFN 11008, vocab 32000)",
            "head": "medusa: 4 heads x K=2 residual SiLU-Linear blocks, shared LM head",
            "tree_nodes": cfg.N, "context": cfg.prompt_len, "batch": cfg.B,
            "acceptance": f"forced, Poisson({FORCED_LAM}) clipped to [{FORCED_LO},{FORCED_HI}]",
            "l2": "inputs larger than L2 (13.5 GB of weights streamed per step)"}


def algorithmic_bytes_per_step(cfg, context: float) -> dict:
    """Bytes that must move once per step: every weight matrix once, plus the KV context."""
    shapes = weight_shapes(cfg)
    layer = sum(int(np.prod(s)) for n, s in shapes.items() if n.startswith("layers.0.") and len(s) == 2) * 2
    lm = cfg.V * cfg.H * 2
    heads = sum(int(np.prod(s)) for n, s in shapes.items() if n.startswith("medusa.") and len(s) == 2) * 2
    kv = cfg.L * cfg.B * context * cfg.n_heads * cfg.head_dim * 2 * 2
    return {"verify_weights": cfg.L * layer + lm, "draft_weights": heads + lm, "kv": kv}


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 8 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 8 and r[1].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) >= 8:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def reduce_over_ranks(times_ms, counts, dist=None, device="cpu"):
    """Whole-job figures from per-rank ones: MAX of the times, SUM of the counts (replicas)."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(v) for v in t], [float(v) for v in n]


# ------------------------------------------------------------------------------------------------
def run_koala(args):
    from paper_2408_08146_b200 import Koala

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=torch.device(dev))
    K, W = args.steps, args.warmup
    extra = 8
    cfg = workload(W + 2 * K + 2 * extra + 4)
    store = WeightStore(cfg, dev)
    eng = Koala(cfg, store.tensors, static_tree=medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk), device=dev)
    eng.prefill(prompts(cfg.with_(seed=cfg.seed + rank)), 64)
    n_sched = W + 2 * K + 2 * extra + 4
    sched = forced_lengths(2000 + cfg.seed + rank, n_sched * cfg.B, FORCED_LAM, FORCED_LO, FORCED_HI).reshape(n_sched, cfg.B)
    sched_host = torch.from_numpy(sched).pin_memory()
    sched_dev = sched_host.to(dev)
    stream = torch.cuda.current_stream()
    it = 0

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W):
        eng.step(sched_dev[it]); it += 1
    # ---- timed region: K steps, inputs resident in HBM
    barrier()
    s_before = eng.seq_len.clone()
    launches_before = eng.launch_count()
    print(f"[bench] library kernels launched before the timed region: {launches_before}", file=sys.stderr)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        barrier()
        e0.record(stream)
        for _ in range(K):
            eng.step(sched_dev[it]); it += 1
        e1.record(stream)
        barrier()
    ms = e0.elapsed_time(e1)
    launches = eng.launch_count() - launches_before
    tokens = int((eng.seq_len - s_before).sum().item())
    assert tokens == int(sched[W:W + K].sum()), "accepted lengths do not follow the forced schedule"
    assert eng.device_status() == 0, "device status word is set"
    mean_ctx = float(s_before.float().mean().item()) + tokens / (2.0 * cfg.B)
    if args.timed_only:
        print(json.dumps({"metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "steps": K, "warmup": W,
                          "ms_per_step": ms / K, "gpu_launches": launches, "note": "timed-only run"}))
        eng.close()
        return

    # ---- end to end through the public calls with host buffers: per step the forced lengths come
    #      from pinned host memory and the step's tokens are read back to the host
    out_tok_h = torch.zeros(cfg.B, eng.out_stride, dtype=torch.int32).pin_memory()
    out_len_h = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    forced_d = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s_before2 = eng.seq_len.clone()
    f0.record(stream)
    for _ in range(K):
        forced_d.copy_(sched_host[it], non_blocking=True)
        ot, ol = eng.step(forced_d); it += 1
        out_tok_h.copy_(ot, non_blocking=True)
        out_len_h.copy_(ol, non_blocking=True)
        stream.synchronize()
    f1.record(stream)
    barrier()
    ms_e2e = f0.elapsed_time(f1)
    tokens_e2e = int((eng.seq_len - s_before2).sum().item())

    # ---- per-call latency (events between the calls) and per-kernel-class time (instrumented pass)
    calls = {"draft": 0.0, "expand": 0.0, "verify": 0.0, "accept": 0.0}
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    for _ in range(extra):
        f = sched_dev[it]; it += 1
        evs[0].record(stream); eng.koala_draft(0)
        evs[1].record(stream); eng.koala_expand_tree(0)
        evs[2].record(stream); eng.koala_verify(None)
        evs[3].record(stream); eng.koala_accept(f)
        evs[4].record(stream); stream.synchronize()
        for i, n in enumerate(calls):
            calls[n] += evs[i].elapsed_time(evs[i + 1]) / extra
    eng.set_timing(True)
    for _ in range(extra):
        eng.step(sched_dev[it]); it += 1
    tim = eng.timing()
    eng.set_timing(False)
    peak, peak_src = measured_peaks()
    g = tim["gemm_tc"]
    achieved = g["bytes"] / (g["ms"] * 1e-3) / 1e9 if g["ms"] > 0 else 0.0
    ab = algorithmic_bytes_per_step(cfg, mean_ctx)

    # ---- reduce over ranks
    t, n = reduce_over_ranks([ms, ms_e2e], [tokens, tokens_e2e, launches], dist, dev)
    ms_max, ms_e2e_max = t[0], t[1]
    line = {
        "metric": METRIC, "value": float(n[0]) / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_desc(cfg),
        "clocks": clocks.summary(),
        "e2e": {"value": float(n[1]) / (ms_e2e_max * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": 4 * cfg.B, "d2h_bytes_per_step": 4 * cfg.B * (eng.out_stride + 1)},
        "gpu_launches": int(n[2]),
        "roofline": {"bound": "hbm", "kernel": "gemm_tc_kernel (all weight-streaming GEMMs of a step)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": f"of {peak_src}",
                     # DRAM bytes per launch (average over a step's GEMM launches): algorithmic bytes x 1.03, the
                     # read ratio ncu measured on the O-projection and gate/up launches
                     # (profiles/ncu_gemm_tc_kernel_t7_o_gateup.md); traffic grows with the weight bytes
                     "traffic": 1.03 * g["bytes"] / max(g["launches"], 1),
                     "algorithmic_bytes_per_launch": g["bytes"] / max(g["launches"], 1),
                     "launches_per_step": g["launches"] / extra, "ms_per_step_in_kernel": g["ms"] / extra},
        "step_roofline": {"algorithmic_bytes_per_step": ab, "achieved_GBps":
                          (ab["verify_weights"] + ab["draft_weights"] + ab["kv"]) / (ms_max / K * 1e-3) / 1e9,
                          "frac_of_peak": (ab["verify_weights"] + ab["draft_weights"] + ab["kv"])
                          / (ms_max / K * 1e-3) / 1e9 / peak},
        "calls_ms": calls,
        "kernel_classes": {k: {"ms_per_step": v["ms"] / extra, "launches_per_step": v["launches"] / extra}
                           for k, v in tim.items()},
        "mean_accepted_len": float(n[0]) / (K * cfg.B * world),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_oracle_leg(cfg, store, steps=1, warmup=1)
    eng.close()
    del eng
    if rank == 0 and world == 1:
        line["autoregressive"] = autoregressive_leg(cfg, store, dev, steps=max(K, 8))
        line["autoregressive"]["speedup_ratio_at_forced_acceptance"] = line["value"] / line["autoregressive"]["value"]
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def autoregressive_leg(cfg, store, dev, steps: int):
    """Vanilla autoregressive decoding with the same target (the denominator of the paper's wall-time
    speed-up ratio, Section 4.1): every step verifies a one-node tree and accepts its bonus token."""
    from paper_2408_08146_b200 import Koala
    ar_cfg = cfg.with_(name=cfg.name + "_ar", N=1, S_max=cfg.prompt_len + steps + 80)
    one = np.asarray([-1], np.int32), np.asarray([0], np.int32), np.asarray([0], np.int32)
    eng = Koala(ar_cfg, store.tensors, static_tree=one, device=dev)
    pr = prompts(cfg)
    # one-node chains: the prompt is ingested token by token here, so seed the cache length instead
    eng.seq_len.fill_(cfg.prompt_len)
    bufs = eng.buffers()
    par = torch.full((cfg.B, 1), -1, dtype=torch.int32, device=dev)
    n1 = torch.ones(cfg.B, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        eng.koala_verify((bufs["root_tok"].view(cfg.B, 1), par, n1, 1))
        eng.koala_accept(None)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert eng.device_status() == 0
    eng.close()
    return {"value": cfg.B / (ms * 1e-3), "unit": UNIT, "ms_per_token": ms, "steps": steps,
            "note": "same target, one-node tree per step, cache length seeded at the prompt length"}


# ------------------------------------------------------------------------------------------------
def cpu_oracle_leg(cfg, store, steps: int, warmup: int):
    """Times the oracle, as it stands, on the host cores: whole iterations (draft, expansion,
    verification, acceptance) at the benchmark's shapes from seeded synthetic caches of the same
    context length (the oracle's cost does not depend on the cache contents)."""
    from oracle.koala_oracle import KoalaOracle
    from threadpoolctl import threadpool_info

    t0 = time.time()
    cache = {}

    def weight(name):
        if name not in cache:
            cache[name] = store.host(name, np.float32)
        return cache[name]

    for name in store.tensors:
        weight(name)
    st = medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk)
    orc = KoalaOracle(cfg, weight, dtype=np.float32, static_tree=st)
    S = cfg.prompt_len
    dev = store.device
    for name, caches in (("target_k", orc.target_k), ("target_v", orc.target_v)):
        for l in range(cfg.L):
            kv = normal_tensor(2000 + cfg.seed, f"{name}.{l}", (cfg.B, S, cfg.n_heads, cfg.head_dim), 1.0, 0.0,
                               torch.bfloat16, dev).float().cpu().numpy()
            for b in range(cfg.B):
                caches[l][b][:S] = kv[b]
    hid = normal_tensor(3000 + cfg.seed, "pend_hid", (cfg.B, 1, cfg.H), 1.0, 0.0, torch.float32, dev).cpu().numpy()
    root = uniform_ints(3000 + cfg.seed, "root_tok", cfg.B, 0, cfg.V)
    for b in range(cfg.B):
        orc.seq_len[b] = S
        orc.pend_hid[b] = hid[b]
        orc.pend_tok[b] = []
        orc.root_tok[b] = int(root[b])
    sched = forced_lengths(2000 + cfg.seed, (steps + warmup) * cfg.B, FORCED_LAM, FORCED_LO, FORCED_HI).reshape(-1, cfg.B)
    setup_s = time.time() - t0
    for i in range(warmup):
        orc.step(list(sched[i]))
    tokens = 0
    t1 = time.time()
    for i in range(warmup, warmup + steps):
        _, lens = orc.step(list(sched[i]))
        tokens += sum(lens)
    dt = time.time() - t1
    threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    return {"value": tokens / dt, "unit": UNIT, "cores": threads, "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{steps} whole iteration(s) (draft, expand, verify of {cfg.N} nodes through {cfg.L} layers, accept) "
                      f"at context {S} from synthetic caches, fp32 numpy, after {warmup} warm-up; {tokens} tokens",
            "ms_per_step": dt / steps * 1e3, "setup_s": setup_s}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, W = args.steps, args.warmup
    cfg = workload(W + K + 4)
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    store = WeightStore(cfg, dev)
    leg = cpu_oracle_leg(cfg, store, steps=K, warmup=W)
    line = {"impl": "reference", "metric": METRIC, "value": leg["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": W,
            "ms_per_step": leg["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_desc(cfg),
            "cpu_baseline": {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": leg["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=24)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="koala", choices=["koala", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--timed-only", action="store_true",
                    help="only the warm-up and the timed steps (for profiler launch lists): no end-to-end, "
                         "per-call or per-kernel passes, no CPU baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_koala(args)


if __name__ == "__main__":
    main()
