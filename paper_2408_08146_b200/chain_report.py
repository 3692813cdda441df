"""The paper's three metrics (Section 4.1) from the library's own counters, with chain drafts.

    python -m paper_2408_08146_b200.chain_report [--layers 32] [--K 1] [--depth 3] [--iters 40] [--sampled]

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


def sampled_step(eng, cfg, u):
    """One iteration with sampled drafts and speculative-sampling acceptance (Section 2.2)."""
    eng.koala_set_sampling(u[0])
    for p in range(cfg.D):
        eng.koala_draft(p)
        eng.koala_expand_tree(p)
    eng.koala_verify(None)
    return eng.koala_accept_sampled(u[1], u[2])


def timed_steps(eng, n, cfg=None, uniforms=None):
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0
    e0.record()
    lens = []
    for i in range(n):
        if uniforms is not None:
            lens.append(sampled_step(eng, cfg, uniforms[i])[1].clone())
        else:
            lens.append(eng.step()[1].clone())
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
    ap.add_argument("--sampled", action="store_true",
                    help="sampled drafts + speculative-sampling acceptance (temperature 1) instead of greedy")
    args = ap.parse_args()
    d = args.depth
    need = args.context + (args.iters + 8) * (d + 1) + 64
    chain = T7_EAGLE.with_(L=args.layers, K=args.K, D=d, topk=1, N=d + 1, prompt_len=args.context,
                           S_max=((need + 127) // 128) * 128)
    store = WeightStore(chain, "cuda:0")
    eng = Koala(chain, store.tensors)
    eng.prefill(prompts(chain), chain.N)
    uniforms = None
    if args.sampled:
        g = torch.Generator(device="cuda:0").manual_seed(1)
        uniforms = [(torch.rand(1, d, device="cuda:0", generator=g), torch.rand(1, d, device="cuda:0", generator=g),
                     torch.rand(1, device="cuda:0", generator=g)) for _ in range(args.iters + 3)]
    for i in range(3):
        sampled_step(eng, chain, uniforms[args.iters + i]) if args.sampled else eng.step()
    eng.koala_accept_stats(1, reset=True)
    ms, toks = timed_steps(eng, args.iters, chain, uniforms)
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
    print("sampled drafts, speculative-sampling acceptance" if args.sampled else "greedy drafts, greedy acceptance")
    print(f"chain drafts, depth {d}, K = {args.K}, {args.layers} layers, context {args.context}, {args.iters} iterations")
    print(f"  average acceptance length l = {ell:.3f} tokens per target forward")
    for n in range(1, d + 1):
        a = hits[n - 1] / trials[n - 1] if trials[n - 1] else float('nan')
        print(f"  {n}-alpha = {a:.3f}  ({hits[n - 1]} of {trials[n - 1]})")
    print(f"  {ms / args.iters:.3f} ms per iteration = {spec_ms_per_tok:.3f} ms per token; one token per step: {ar_ms:.3f} ms")
    print(f"  wall-time speed-up ratio = {ar_ms / spec_ms_per_tok:.3f}")


if __name__ == "__main__":
    main()
