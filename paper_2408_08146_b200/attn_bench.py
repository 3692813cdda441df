"""Times the tree-masked attention kernel on a two-layer slice of the 7B shape.

    python -m paper_2408_08146_b200.attn_bench [--rows 64] [--context 512] [--batch 1] [--iters 20]
                                               [--mma-sync]

Runs `koala_verify` on a random caller tree over zero-filled caches of the given context length
and reports the device time between the events that bracket each attention launch
(`KOALA_OPT_TIMING`, which serialises the launches), with the K/V bytes that launch reads.
`--mma-sync` selects the mma.sync kernel for every row count (the default picks the tcgen05
kernel from 16 rows per sequence up).  The slice keeps memory small (about 1 GB), which is what an
`ncu` capture of this kernel wants.  Run from the repository root.
"""
from __future__ import annotations

import argparse
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import T7_EAGLE, reduced  # noqa: E402
from workloads.generate import WeightStore  # noqa: E402

from . import Koala, binding  # noqa: E402
from .sweep import random_tree  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=64)
    ap.add_argument("--context", type=int, default=512)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--mma-sync", action="store_true")
    ap.add_argument("--chunks", type=int, default=0, help="key chunks per (sequence, head): 1, 2, 4, 8; 0 = automatic")
    ap.add_argument("--l2-ahead", type=int, default=-1, help="K/V tiles requested into L2 ahead of the ring (-1 = the library's default)")
    args = ap.parse_args()
    lib = binding.load_library()
    if args.mma_sync:
        lib.koala_set_tuning(9, 1 << 20)
    lib.koala_set_tuning(12, args.chunks)
    if args.l2_ahead >= 0:
        lib.koala_set_tuning(19, args.l2_ahead)
    n = args.rows
    cfg = reduced(T7_EAGLE, 2, K=1, N=n, B=args.batch, D=min(5, max(1, n - 1)), V=4096,
                  S_max=((args.context + n + 127) // 128) * 128)
    store = WeightStore(cfg, "cuda:0")
    eng = Koala(cfg, store.tensors)
    eng.seq_len.fill_(args.context)
    tree = random_tree(cfg, n, 77)
    for _ in range(3):
        eng.koala_verify(tree)
    torch.cuda.synchronize()
    eng.set_timing(True)
    for _ in range(args.iters):
        eng.koala_verify(tree)
    t = eng.timing()["attention"]
    eng.set_timing(False)
    assert eng.device_status() == 0
    us = 1e3 * t["ms"] / t["launches"]
    kv = args.batch * cfg.n_heads * (args.context + n) * cfg.head_dim * 2 * 2
    print(f"attention (chunks {args.chunks or 'auto'}): rows {n} x batch {args.batch}, context {args.context}: {us:.2f} us per launch "
          f"({t['launches']} launches, event-bracketed), {kv / 1e6:.2f} MB of K/V per launch = {kv / us / 1e3:.0f} GB/s")
    eng.close()


if __name__ == "__main__":
    main()
