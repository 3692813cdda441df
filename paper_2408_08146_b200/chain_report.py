"""The paper's three metrics (Section 4.1) from the library's own counters, with chain drafts.

    python -m paper_2408_08146_b200.chain_report [--layers 32] [--K 1] [--depth 3] [--iters 40]

Runs an EAGLE-style head on the 7B shape in chain mode (top-1 per level, a tree of depth+1 nodes,
no tree attention needed), free-running with greedy acceptance, and prints
  * the average acceptance length l (tokens per target forward, bonus included),
  * n-alpha for n = 1 .. depth (`koala_accept_stats`: hits / trials per chain position),
  * the wall-time ratio against the same target decoding one token per step (a one-node tree).
The weights are random (there are no trained heads here), so the head agrees with the target
only by chance: expect l = 1, n-alpha = 0 and a ratio below 1.  The point is the mechanism: the
same three numbers come out for real weights.  Run from the repository root.
"""
from __future__ import annotations

import argparse
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import T7_EAGLE  # noqa: E402
from workloads.generate import WeightStore, prompts  # noqa: E402

from . import Koala  # noqa: E402


def timed_steps(eng, n):
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0
    e0.record()
    lens = []
    for _ in range(n):
        lens.append(eng.step()[1])
    e1.record()
    torch.cuda.synchronize()
    for ln in lens:
        total += int(ln.sum().item())
    return e0.elapsed_time(e1), total


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--K", type=int, default=1)
    ap.add_argument("--depth", type=int, default=3)
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--context", type=int, default=256)
    args = ap.parse_args()
    d = args.depth
    need = args.context + (args.iters + 8) * (d + 1) + 64
    chain = T7_EAGLE.with_(L=args.layers, K=args.K, D=d, topk=1, N=d + 1, prompt_len=args.context,
                           S_max=((need + 127) // 128) * 128)
    store = WeightStore(chain, "cuda:0")
    eng = Koala(chain, store.tensors)
    eng.prefill(prompts(chain), chain.N)
    for _ in range(3):
        eng.step()
    eng.koala_accept_stats(1, reset=True)
    ms, toks = timed_steps(eng, args.iters)
    hits, trials = eng.koala_accept_stats(d)
    assert eng.device_status() == 0
    eng.close()
    # the same target, one token per step: a one-node tree whose token is the last bonus token;
    # the cache length is seeded instead of ingesting the prompt token by token
    ar = chain.with_(D=1, N=1, S_max=((args.context + args.iters + 80 + 127) // 128) * 128)
    eng = Koala(ar, store.tensors)
    eng.seq_len.fill_(args.context)
    bufs = eng.buffers()
    par = torch.full((1, 1), -1, dtype=torch.int32, device="cuda:0")
    n1 = torch.ones(1, dtype=torch.int32, device="cuda:0")
    stream = torch.cuda.current_stream()

    def ar_step():
        eng.koala_verify((bufs["root_tok"].view(1, 1), par, n1, 1))
        eng.koala_accept(None)

    for _ in range(3):
        ar_step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.iters):
        ar_step()
    e1.record(stream)
    torch.cuda.synchronize()
    ar_ms = e0.elapsed_time(e1) / args.iters
    assert eng.device_status() == 0
    eng.close()
    ell = toks / args.iters
    spec_ms_per_tok = ms / max(1, toks)
    print(f"chain drafts, depth {d}, K = {args.K}, {args.layers} layers, context {args.context}, {args.iters} iterations")
    print(f"  average acceptance length l = {ell:.3f} tokens per target forward")
    for n in range(1, d + 1):
        a = hits[n - 1] / trials[n - 1] if trials[n - 1] else float('nan')
        print(f"  {n}-alpha = {a:.3f}  ({hits[n - 1]} of {trials[n - 1]})")
    print(f"  {ms / args.iters:.3f} ms per iteration = {spec_ms_per_tok:.3f} ms per token; one token per step: {ar_ms:.3f} ms")
    print(f"  wall-time speed-up ratio = {ar_ms / spec_ms_per_tok:.3f}")


if __name__ == "__main__":
    main()
