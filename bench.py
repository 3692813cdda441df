#!/usr/bin/env python
"""Benchmark of the draft-then-verify step (speculative decoding with K-layer draft heads).

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A step is one whole iteration of the hot path (draft passes, tree expansion, verification of the
whole tree in one target forward, greedy acceptance + KV compaction) over one batch.

Headline workload (the largest configuration that runs on one GPU): the 13B-shaped target in bf16
with a 2-layer EAGLE-style head, batch 4 with ragged prompts of 512..2048 tokens, dynamic 64-node
trees (depth 5, top-10).  Weights are seeded N(0, 0.02), prompts seeded uniform token ids.  Random
heads accept nothing, so the accepted length of each step is forced from a seeded schedule
(Poisson(3) clipped to [1, 6]).

On one GPU the same line also carries, as named legs, the 7B-shaped configurations (Medusa-style
heads with the static 64-node tree at context 512; EAGLE-style head with K = 1, 2, 4 at context
1024), draft latency against K, verify latency against the tree size, the library's own
one-token-per-step loop, and the CPU oracle timed on the host cores.

Prints one JSON line.  With N > 1 every rank runs an independent replica of the headline workload
(sequences share only read-only weights, so there is no data-path collective) and the value is the
whole job's.  `--impl reference` times the CPU oracle on the host cores instead (a deliberately
slow baseline).
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

from workloads import T13_EAGLE, T7_EAGLE, T7_MEDUSA  # noqa: E402
from workloads.configs import EAGLE  # noqa: E402
from workloads.generate import (WeightStore, forced_lengths, medusa_static_tree, prompt_lengths, prompts,  # noqa: E402
                                normal_tensor, uniform_ints)

METRIC = "spec_decode_tokens_per_s"
UNIT = "tokens/s"
FORCED_LAM = 3.0
HEADLINE = T13_EAGLE
# DRAM traffic of the dominant launch from its ncu capture (one launch of gemm_tc_pair_kernel on the
# 13B gate+up shape at 256 tokens, a 1.4 GB case: dram__bytes_read.sum + dram__bytes_write.sum), used
# to scale the step's weight bytes per GEMM launch to DRAM bytes per launch: the traffic is the
# weights once (1.03 x) plus one write-back of the fp32 partial sums, both proportional to the matrix.
NCU_DRAM_BYTES = 291.5e6 + 28.2e6
NCU_ALGORITHMIC_BYTES = 283.1e6
NCU_SOURCE = ("scaled from one ncu capture of the dominant launch (gemm_tc_pair_kernel, 13B gate+up at 256 tokens: "
              "319.7 MB of DRAM traffic for 283.1 MB of weights; profiles/ncu_gemm_tc_pair_kernel_t13_gateup_256tokens.md) "
              "by the weight bytes per launch of this step")


def forced_range(cfg):
    """Accepted lengths are clipped to [1, D + 1]: at most D drafted tokens plus the bonus token."""
    return 1, cfg.D + 1


def with_capacity(cfg, steps_total: int):
    """KV capacity for the longest prompt, every step's growth and one tree."""
    s_max = cfg.prompt_len + steps_total * (cfg.D + 1) + cfg.N + 64
    return cfg.with_(S_max=(s_max + 127) // 128 * 128)


def workload_desc(cfg):
    head = (f"EAGLE-style: fc(2H->H) + K={cfg.K} decoder layers, dynamic tree depth {cfg.D} top-{cfg.topk}"
            if cfg.head_kind == EAGLE else
            f"Medusa-style: {cfg.n_medusa_heads} heads x K={cfg.K} residual SiLU-Linear blocks, shared LM head, static tree")
    ctx = (f"ragged, uniform in [{cfg.prompt_len_min}, {cfg.prompt_len}]" if cfg.prompt_len_min > 0 else cfg.prompt_len)
    lo, hi = forced_range(cfg)
    return {"workload": cfg.name,
            "target": f"Llama-shaped: {cfg.L} layers, hidden {cfg.H}, {cfg.n_heads}x{cfg.head_dim} heads, FFN {cfg.F}, vocab {cfg.V}",
            "head": head, "tree_nodes": cfg.N, "context": ctx, "batch": cfg.B,
            "acceptance": f"forced, Poisson({FORCED_LAM}) clipped to [{lo},{hi}]",
            "l2": "inputs larger than L2 (every weight matrix is streamed once per step)"}


def algorithmic_work(cfg, context: float) -> dict:
    """What must move / be computed once per step: every weight matrix once per forward that uses it,
    plus the KV context; flops of the dense contractions (2 per weight per row)."""
    H, F, V = cfg.H, cfg.F, cfg.V
    layer = (4 * H * H + 3 * H * F) * 2
    lm = V * H * 2
    kv_tok = cfg.B * context * H * 2 * 2                       # K and V bytes of one layer
    rows = cfg.B * cfg.N
    verify_w = cfg.L * layer + lm
    if cfg.head_kind == EAGLE:
        pass_w = 2 * H * H * 2 + cfg.K * layer + lm
        draft_w = cfg.D * pass_w
        draft_kv = cfg.D * cfg.K * kv_tok
        draft_flops = 2.0 * (pass_w / 2) * cfg.B * (1 + (cfg.D - 1) * cfg.topk)
    else:
        draft_w = cfg.n_medusa_heads * cfg.K * H * H * 2 + lm
        draft_kv = 0.0
        draft_flops = 2.0 * (draft_w / 2) * cfg.B * cfg.n_medusa_heads
    return {"verify_weights": verify_w, "draft_weights": draft_w, "kv": cfg.L * kv_tok + draft_kv,
            "flops": 2.0 * (verify_w / 2) * rows + draft_flops}


def step_roofline(cfg, context: float, ms_per_step: float, peaks: dict) -> dict:
    w = algorithmic_work(cfg, context)
    nbytes = w["verify_weights"] + w["draft_weights"] + w["kv"]
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_tc = w["flops"] / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    bound_ms = max(t_hbm, t_tc)
    return {"algorithmic_bytes_per_step": nbytes, "algorithmic_flops_per_step": w["flops"],
            "ideal_ms_hbm": t_hbm, "ideal_ms_tensor": t_tc,
            # bf16 activations enter the MMAs as a value + residual pair: twice the algorithmic flops are issued
            "ideal_ms_tensor_issued": 2.0 * t_tc if cfg.dtype == 1 else t_tc, "bound": "hbm" if t_hbm >= t_tc else "tensor",
            "achieved_GBps": nbytes / (ms_per_step * 1e-3) / 1e9, "achieved_TFLOPs": w["flops"] / (ms_per_step * 1e-3) / 1e12,
            "frac_of_peak": bound_ms / ms_per_step, "peak_source": f"of {peaks['source']}"}


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


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def reduce_over_ranks(times_ms, counts, dist=None, device="cpu"):
    """Whole-job figures from per-rank ones: MAX of the times, SUM of the counts (replicas)."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(v) for v in t], [float(v) for v in n]


# ------------------------------------------------------------------------------------------------
def make_engine(cfg, store, dev):
    from paper_2408_08146_b200 import Koala
    st = None if cfg.head_kind == EAGLE else medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk)
    return Koala(cfg, store.tensors, static_tree=st, device=dev)


def schedule(cfg, seed, n_steps):
    lo, hi = forced_range(cfg)
    return forced_lengths(seed, n_steps * cfg.B, FORCED_LAM, lo, hi).reshape(n_steps, cfg.B)


class Snapshot:
    """The small per-sequence state a step reads besides the caches (lengths, next root, the rows
    accepted last): restoring it replays the same schedule slice from the same context lengths."""
    NAMES = ("root_tok", "n_pend", "pend_tok", "pend_hid")

    def __init__(self, eng):
        self.eng = eng
        b = eng.buffers()
        self.seq_len = eng.seq_len.clone()
        self.saved = {n: b[n].clone() for n in self.NAMES}

    def restore(self):
        b = self.eng.buffers()
        self.eng.seq_len.copy_(self.seq_len)
        for n in self.NAMES:
            b[n].copy_(self.saved[n])


def timed_steps(eng, sched_dev, start, K, stream, barrier=None, clocks_index=None):
    """K steps with inputs resident in HBM, CUDA events on the launching stream."""
    sync = barrier or torch.cuda.synchronize
    sync()
    before = eng.seq_len.clone()
    launches_before = eng.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(clocks_index) if clocks_index is not None else None
    if sampler:
        sampler.__enter__()
    sync()
    e0.record(stream)
    for i in range(K):
        eng.step(sched_dev[start + i])
    e1.record(stream)
    sync()
    if sampler:
        sampler.__exit__()
    ms = e0.elapsed_time(e1)
    tokens = int((eng.seq_len - before).sum().item())
    ctx = float(before.float().mean().item()) + tokens / (2.0 * eng.cfg.B)
    return {"ms": ms, "tokens": tokens, "launches": eng.launch_count() - launches_before, "mean_context": ctx,
            "clocks": sampler.summary() if sampler else None}


def per_call_ms(eng, sched_dev, start, n, stream):
    """Average device time of each of the five calls (events between the calls)."""
    cfg = eng.cfg
    passes = cfg.D if cfg.head_kind == EAGLE else 1
    calls = {"draft": 0.0, "expand": 0.0, "verify": 0.0, "accept": 0.0}
    draft_pass = np.zeros(passes)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(2 * passes + 3)]
    for i in range(n):
        for p in range(passes):
            evs[2 * p].record(stream); eng.koala_draft(p)
            evs[2 * p + 1].record(stream); eng.koala_expand_tree(p)
        evs[2 * passes].record(stream); eng.koala_verify(None)
        evs[2 * passes + 1].record(stream); eng.koala_accept(sched_dev[start + i])
        evs[2 * passes + 2].record(stream); stream.synchronize()
        for p in range(passes):
            d = evs[2 * p].elapsed_time(evs[2 * p + 1])
            calls["draft"] += d / n
            draft_pass[p] += d / n
            calls["expand"] += evs[2 * p + 1].elapsed_time(evs[2 * p + 2]) / n
        calls["verify"] += evs[2 * passes].elapsed_time(evs[2 * passes + 1]) / n
        calls["accept"] += evs[2 * passes + 1].elapsed_time(evs[2 * passes + 2]) / n
    calls["draft_per_pass"] = [float(x) for x in draft_pass]
    return calls


def leg(cfg, store, dev, steps, warmup, peaks, seed_off=0):
    """One named configuration: prompt ingestion, warm-up, `steps` timed steps, per-call times."""
    extra = 4
    n_sched = warmup + steps + extra + 2
    cfg = with_capacity(cfg, n_sched)
    eng = make_engine(cfg, store, dev)
    eng.prefill(prompts(cfg), 64)
    sched = schedule(cfg, 2000 + cfg.seed + seed_off, n_sched)
    sched_dev = torch.from_numpy(sched).to(dev)
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        eng.step(sched_dev[i])
    r = timed_steps(eng, sched_dev, warmup, steps, stream)
    assert r["tokens"] == int(sched[warmup:warmup + steps].sum()), "accepted lengths do not follow the forced schedule"
    calls = per_call_ms(eng, sched_dev, warmup + steps, extra, stream)
    assert eng.device_status() == 0, "device status word is set"
    eng.close()
    ms_step = r["ms"] / steps
    out = {"config": workload_desc(cfg), "steps": steps, "warmup": warmup, "ms_per_step": ms_step,
           "value": r["tokens"] / (r["ms"] * 1e-3), "unit": UNIT, "mean_accepted_len": r["tokens"] / (steps * cfg.B),
           "gpu_launches": r["launches"], "calls_ms": calls,
           "step_roofline": step_roofline(cfg, r["mean_context"], ms_step, peaks)}
    w = algorithmic_work(cfg, r["mean_context"])
    out["verify_frac_of_hbm_peak"] = (w["verify_weights"] + cfg.L * cfg.B * r["mean_context"] * cfg.H * 4) \
        / (calls["verify"] * 1e-3) / 1e9 / peaks["hbm_gbs"]
    out["draft_frac_of_hbm_peak"] = (w["draft_weights"] + (w["kv"] - cfg.L * cfg.B * r["mean_context"] * cfg.H * 4)) \
        / (calls["draft"] * 1e-3) / 1e9 / peaks["hbm_gbs"]
    return out


# ------------------------------------------------------------------------------------------------
def run_koala(args):
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
    extra = 6
    peaks = measured_peaks()
    n_sched = W + K + 2 * extra + 4
    cfg = with_capacity(HEADLINE, n_sched)
    store = WeightStore(cfg, dev)
    eng = make_engine(cfg, store, dev)
    eng.prefill(prompts(cfg.with_(seed=cfg.seed + rank)), 64)
    sched = schedule(cfg, 2000 + cfg.seed + rank, n_sched)
    sched_host = torch.from_numpy(sched).pin_memory()
    sched_dev = sched_host.to(dev)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(W):
        eng.step(sched_dev[i])
    # ---- timed region: K steps, inputs resident in HBM
    barrier()
    snap = Snapshot(eng)
    print(f"[bench] library kernels launched before the timed region: {eng.launch_count()}", file=sys.stderr)
    r = timed_steps(eng, sched_dev, W, K, stream, barrier, local)
    ms, tokens, launches = r["ms"], r["tokens"], r["launches"]
    assert tokens == int(sched[W:W + K].sum()), "accepted lengths do not follow the forced schedule"
    assert eng.device_status() == 0, "device status word is set"
    if args.timed_only:
        print(json.dumps({"metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "steps": K, "warmup": W,
                          "ms_per_step": ms / K, "gpu_launches": launches, "note": "timed-only run"}))
        eng.close()
        return

    # ---- end to end through the public calls with host buffers, over the SAME schedule slice from
    #      the same context lengths: per step the forced lengths come from pinned host memory and
    #      the step's tokens and lengths are read back to the host
    snap.restore()
    out_tok_h = torch.zeros(cfg.B, eng.out_stride, dtype=torch.int32).pin_memory()
    out_len_h = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    forced_d = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s_before2 = eng.seq_len.clone()
    f0.record(stream)
    for i in range(K):
        forced_d.copy_(sched_host[W + i], non_blocking=True)
        ot, ol = eng.step(forced_d)
        out_tok_h.copy_(ot, non_blocking=True)
        out_len_h.copy_(ol, non_blocking=True)
        stream.synchronize()
    f1.record(stream)
    barrier()
    ms_e2e = f0.elapsed_time(f1)
    tokens_e2e = int((eng.seq_len - s_before2).sum().item())
    assert tokens_e2e == tokens

    # ---- per-call latency (events between the calls) and per-kernel-class time (instrumented pass)
    it = W + K
    calls = per_call_ms(eng, sched_dev, it, extra, stream)
    it += extra
    eng.set_timing(True)
    for i in range(extra):
        eng.step(sched_dev[it + i])
    tim = eng.timing()
    eng.set_timing(False)
    g = tim["gemm_tc"]
    achieved = g["bytes"] / (g["ms"] * 1e-3) / 1e9 if g["ms"] > 0 else 0.0
    g_flops = 2.0 * (g["bytes"] / 2) * cfg.B * cfg.N        # upper bound: every launch at the verify's row count

    # ---- reduce over ranks
    t, n = reduce_over_ranks([ms, ms_e2e], [tokens, tokens_e2e, launches], dist, dev)
    ms_max, ms_e2e_max = t[0], t[1]
    sr = step_roofline(cfg, r["mean_context"], ms_max / K, peaks)
    line = {
        "metric": METRIC, "value": float(n[0]) / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_desc(cfg),
        "clocks": r["clocks"],
        "e2e": {"value": float(n[1]) / (ms_e2e_max * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e_max / K,
                "tokens": int(n[1]), "schedule": "the timed region's slice, replayed from the same context lengths",
                "h2d_bytes_per_step": 4 * cfg.B, "d2h_bytes_per_step": 4 * cfg.B * (eng.out_stride + 1)},
        "gpu_launches": int(n[2]),
        "roofline": {"bound": "hbm", "kernel": "gemm_tc_pair_kernel + gemm_tc_kernel (all weight-streaming GEMMs of a step: the CTA-pair form "
                               "for the verification's 256 rows, the one-CTA form for the draft passes and the LM head)",
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": f"of {peaks['source']}",
                     "traffic": g["bytes"] / max(g["launches"], 1) * NCU_DRAM_BYTES / NCU_ALGORITHMIC_BYTES,
                     "traffic_source": NCU_SOURCE,
                     "algorithmic_bytes_per_launch": g["bytes"] / max(g["launches"], 1),
                     "launches_per_step": g["launches"] / extra, "ms_per_step_in_kernel": g["ms"] / extra,
                     "tensor_TFLOPs_upper_bound": g_flops / (g["ms"] * 1e-3) / 1e12 if g["ms"] > 0 else 0.0},
        "step_roofline": sr,
        "calls_ms": calls,
        "kernel_classes": {k: {"ms_per_step": v["ms"] / extra, "launches_per_step": v["launches"] / extra}
                           for k, v in tim.items()},
        "mean_accepted_len": float(n[0]) / (K * cfg.B * world),
    }
    eng.close()
    del eng
    torch.cuda.empty_cache()
    if rank == 0 and world == 1:
        line["autoregressive"] = autoregressive_leg(cfg, store, dev, steps=max(K, 8))
        line["autoregressive"]["speedup_ratio_at_forced_acceptance"] = line["value"] / line["autoregressive"]["value"]
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_leg(HEADLINE, store, steps=1, warmup=0)
    del store
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_legs:
        line.update(other_configurations(dev, peaks, steps=min(K, 12), warmup=3))
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def other_configurations(dev, peaks, steps, warmup):
    """The 7B-shaped configurations as named legs, and the two latency curves of the metric."""
    from paper_2408_08146_b200.sweep import draft_sweep, verify_sweep
    out = {"legs": {}}
    store = WeightStore(T7_MEDUSA, dev)
    out["legs"]["t7_medusa_K2_ctx512"] = leg(T7_MEDUSA, store, dev, steps, warmup, peaks)
    del store
    torch.cuda.empty_cache()
    store = WeightStore(T7_EAGLE.with_(K=4), dev)          # draft layers 0..3: every K below uses a prefix
    for k in (1, 2, 4):
        out["legs"][f"t7_eagle_K{k}_ctx1024"] = leg(T7_EAGLE.with_(K=k, name=f"t7_eagle_bf16_K{k}"), store, dev, steps,
                                                    warmup, peaks)
    with open(os.devnull, "w") as sink:
        stdout, sys.stdout = sys.stdout, sink
        try:
            d = draft_sweep(store, 6, peaks["hbm_gbs"])
            v = verify_sweep(store, 6, peaks["hbm_gbs"], peaks["bf16_tflops_sustained"], T7_EAGLE,
                             [(n, 1024, 1) for n in (16, 32, 64, 128)])
        finally:
            sys.stdout = stdout
    out["draft_ms_vs_K"] = [{"K": r["K"], "ms_per_pass": sum(r["ms_per_pass"]) / len(r["ms_per_pass"]),
                             "ms_per_iteration": r["ms_per_iteration"], "passes": r["passes"], "context": r["context"],
                             "frac_of_hbm_peak": r["frac_measured"]} for r in d]
    out["verify_ms_vs_tree"] = [{"tree_nodes": r["tree"], "context": r["context"], "batch": r["batch"], "ms": r["ms"],
                                 "frac_of_hbm_peak": r["frac_measured"], "bound": r["bound"]} for r in v]
    out["curves_note"] = ("7B-shaped target, bf16, one sequence: draft = EAGLE-style head, 5 passes (draft + expand_tree) "
                          "at context 1024 on a one-layer target; verify = koala_verify of a random caller tree at context 1024")
    return out


def autoregressive_leg(cfg, store, dev, steps: int):
    """Vanilla autoregressive decoding with the same target (the denominator of the paper's wall-time
    speed-up ratio, Section 4.1): every step verifies a one-node tree and accepts its bonus token."""
    from paper_2408_08146_b200 import Koala
    mean_len = int(prompt_lengths(cfg).mean())
    ar_cfg = cfg.with_(name=cfg.name + "_ar", N=1, D=1, topk=1, K=0, S_max=cfg.prompt_len + steps + 80)
    eng = Koala(ar_cfg, store.tensors, device=dev)
    # one-node chains: the prompt would be ingested token by token here, so seed the cache lengths instead
    eng.seq_len.copy_(torch.from_numpy(prompt_lengths(cfg).astype(np.int32)))
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
    return {"value": cfg.B / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps, "mean_context": mean_len,
            "note": "same target and batch, one-node tree per sequence and step, cache lengths seeded at the prompt lengths"}


# ------------------------------------------------------------------------------------------------
def cpu_oracle_leg(cfg, store, steps: int, warmup: int):
    """Times the oracle, as it stands, on the host cores, on a bounded sample of the headline
    workload: whole iterations (draft passes, expansion, verification, acceptance) of sequence 0 of
    the batch at its own context length, from seeded synthetic caches of that length (the oracle's
    cost does not depend on the cache contents).  The oracle handles the sequences of a batch one
    after the other, so its tokens/s is that of one sequence whatever the batch size."""
    from oracle.koala_oracle import KoalaOracle, round_to_bf16
    from threadpoolctl import threadpool_info

    t0 = time.time()
    S = int(prompt_lengths(cfg)[0])
    one = cfg.with_(B=1, prompt_len=S, prompt_len_min=0, S_max=(S + (steps + warmup) * (cfg.D + 1) + cfg.N + 127) // 128 * 128)
    st = None if cfg.head_kind == EAGLE else medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk)
    # The oracle takes its weights as float32 host arrays.  Where the host has the memory they are
    # converted once, before the timed region; otherwise they are handed over tensor by tensor from the
    # device copies inside it (no second full copy on the host).
    import psutil
    need = sum(t.numel() for t in store.tensors.values()) * 4
    cached = psutil.virtual_memory().available > 1.5 * need + (16 << 30)
    host = {}
    if cached:
        for name in store.tensors:
            host[name] = store.host(name, np.float32)
    getter = (lambda name: host[name]) if cached else (lambda name: store.host(name, np.float32))
    orc = KoalaOracle(one, getter, dtype=np.float32, static_tree=st, kv_round=round_to_bf16)
    dev = store.device
    groups = [("target_k", orc.target_k, one.L), ("target_v", orc.target_v, one.L)]
    if cfg.head_kind == EAGLE:
        groups += [("draft_k", orc.draft_k, one.K), ("draft_v", orc.draft_v, one.K)]
    for name, caches, n_layers in groups:
        for l in range(n_layers):
            kv = normal_tensor(2000 + cfg.seed, f"{name}.{l}", (S, one.n_heads, one.head_dim), 1.0, 0.0,
                               torch.bfloat16, dev).float().cpu().numpy()
            caches[l][0][:S] = kv
    hid = normal_tensor(3000 + cfg.seed, "pend_hid", (1, cfg.H), 1.0, 0.0, torch.float32, dev).cpu().numpy()
    root = uniform_ints(3000 + cfg.seed, "root_tok", 1, 0, cfg.V)
    orc.seq_len[0] = S
    orc.pend_hid[0] = hid
    orc.pend_tok[0] = []
    orc.root_tok[0] = int(root[0])
    sched = schedule(one, 2000 + cfg.seed, steps + warmup)
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
            "sample": f"{steps} whole iteration(s) of sequence 0 of the batch of {cfg.B} ({cfg.D} draft passes of the "
                      f"K={cfg.K} head, expansion, verification of {cfg.N} nodes through {cfg.L} layers, acceptance) at its "
                      f"context of {S} tokens from synthetic caches, fp32 numpy, weights "
                      + ("held as float32 host arrays" if cached else "converted from the bf16 device copies inside the timed region")
                      + f", {warmup} warm-up; {tokens} tokens",
            "ms_per_step": dt / steps * 1e3, "setup_s": setup_s}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, W = args.steps, args.warmup
    cfg = HEADLINE
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    store = WeightStore(cfg, dev)
    leg_ = cpu_oracle_leg(cfg, store, steps=K, warmup=W)
    line = {"impl": "reference", "metric": METRIC, "value": leg_["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": W,
            "ms_per_step": leg_["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_desc(with_capacity(cfg, K + W)),
            "cpu_baseline": {k: leg_[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": leg_["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="koala", choices=["koala", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="headline workload only (no 7B legs, no latency curves)")
    ap.add_argument("--timed-only", action="store_true",
                    help="only the warm-up and the timed steps (for profiler launch lists): no end-to-end, "
                         "per-call or per-kernel passes, no CPU baseline, no legs")
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
