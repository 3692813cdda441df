"""Unserialised kernel timeline of one benchmark step (CUPTI through torch.profiler).

    python -m paper_2408_08146_b200.timeline [--layer 9]

Prints, for the library's kernels of one step of the benchmark workload (7B-shaped target,
Medusa-style heads, 64-node tree, context ~512): the span of the step, and per kernel name the sum
of the end-to-end increments (time from the latest end of any earlier kernel to this kernel's
end), which is how much each kernel adds to the critical path with programmatic dependent launch
overlap in place.  Also lists the kernels of one decoder layer with their start and end times.
Run from the repository root.
"""
from __future__ import annotations

import argparse
import os
import re
import sys

import torch
from torch.profiler import ProfilerActivity, profile

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def short(name: str) -> str:
    m = re.search(r"(\w+_kernel)", name)
    return m.group(1) if m else name[:30]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", type=int, default=9)
    args = ap.parse_args()
    import bench
    from workloads.generate import WeightStore, medusa_static_tree, prompts
    from . import Koala

    from workloads import T7_MEDUSA
    cfg = bench.with_capacity(T7_MEDUSA, 100)
    store = WeightStore(cfg, "cuda:0")
    eng = Koala(cfg, store.tensors, static_tree=medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk))
    eng.prefill(prompts(cfg), 64)
    forced = torch.full((cfg.B,), 3, dtype=torch.int32, device="cuda:0")
    for _ in range(5):
        eng.step(forced)
    torch.cuda.synchronize()
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        for _ in range(3):
            eng.step(forced)
        torch.cuda.synchronize()
    ks = sorted([(e.time_range.start, e.time_range.end, e.name) for e in prof.events() if "koala" in e.name])
    first = [i for i, k in enumerate(ks) if "embed_update" in k[2] or "embed_norm" in k[2]]   # one per verify call
    seg = ks[first[1]:first[2]]
    print(f"step span {ks[first[2]][0] - ks[first[1]][0]:.1f} us, {len(seg)} kernels")
    latest, inc = None, {}
    for s, e, n in seg:
        if latest is not None:
            a = inc.setdefault(short(n), [0, 0.0])
            a[0] += 1
            a[1] += max(0.0, e - latest)
        latest = e if latest is None else max(latest, e)
    print("critical-path increments per kernel name:")
    for k, (c, t) in sorted(inc.items(), key=lambda kv: -kv[1][1]):
        print(f"  {k:28s} n={c:4d}  sum {t:8.1f} us  avg {t / c:6.2f} us")
    per_layer = [i for i, k in enumerate(seg) if "tree_attn" in k[2]]      # one attention launch per decoder layer
    if len(per_layer) > args.layer + 1:
        i0, i1 = per_layer[args.layer], per_layer[args.layer + 1]
        t0 = seg[i0][0]
        print(f"kernels of decoder layer {args.layer} (us from the layer's first kernel start):")
        for s, e, n in seg[i0:i1]:
            print(f"  {short(n):28s} start {s - t0:8.2f}  end {e - t0:8.2f}")
    eng.close()


if __name__ == "__main__":
    main()
