"""Times the library's weight-streaming GEMM on the decoder shapes (kernel sweep).

    python -m paper_2408_08146_b200.gemm_bench [--model 7b|13b] [--tokens 64] [--shapes qkv,o,...]
                                               [--splits 0,1,3] [--stages 0] [--plain] [--iters 20] [--tune key=value,...]

Prints, per shape and split-K factor, the mean time of one call (CUDA events around `iters`
back-to-back calls that rotate over enough weight copies to defeat the L2) and the weight bytes
per second.  With a split > 1 the figure includes the small kernel that sums the partials.
"""
from __future__ import annotations

import argparse

import torch

from . import binding

MODELS = {"7b": dict(H=4096, F=11008, V=32000), "13b": dict(H=5120, F=13824, V=32000)}


def shapes_of(model: str):
    m = MODELS[model]
    H, F, V = m["H"], m["F"], m["V"]
    return {"qkv": (3 * H, H), "o": (H, H), "gateup": (2 * F, H), "down": (H, F), "lm": (V, H),
            "fc": (H, 2 * H), "res": (H, H)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="7b", choices=sorted(MODELS))
    ap.add_argument("--tokens", type=int, default=64)
    ap.add_argument("--shapes", default="qkv,o,gateup,down,lm")
    ap.add_argument("--splits", default="0")
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--plain", action="store_true", help="plain bf16 activations instead of value+residual pairs")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--tune", default="", help="tuning keys of koala_set_tuning, e.g. 2=4,3=1")
    args = ap.parse_args()
    lib = binding.load_library()
    dev = "cuda:0"
    M = args.tokens
    pair = 0 if args.plain else 1
    rows = lib.koala_gemm_x_rows(M, pair)
    lib.koala_set_tuning(1, args.stages)
    for kv in filter(None, args.tune.split(",")):
        k, v = kv.split("=")
        lib.koala_set_tuning(int(k), int(v))
    st = torch.cuda.current_stream().cuda_stream
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for name in args.shapes.split(","):
        N, K = shapes_of(args.model)[name]
        nbuf = max(2, int(1.5e9 // (N * K * 2)))
        Ws = [torch.randn(N, K, device=dev, dtype=torch.bfloat16) * 0.02 for _ in range(nbuf)]
        xh = torch.randn(rows, K, device=dev, dtype=torch.bfloat16)
        xl = (torch.randn(rows, K, device=dev) * 0.003).to(torch.bfloat16)
        y = torch.empty(M, N, device=dev)
        nb = lib.koala_gemm_scratch_bytes(M, N, K)
        scratch = torch.empty(nb, dtype=torch.uint8, device=dev)
        for split in [int(s) for s in args.splits.split(",")]:
            def run(i):
                rc = lib.koala_gemm_bf16(xh.data_ptr(), xl.data_ptr() if pair else None, Ws[i % nbuf].data_ptr(),
                                         y.data_ptr(), N, M, N, K, scratch.data_ptr(), nb, 1, split, st,
                                         status.data_ptr())
                assert rc == 0, rc
            for i in range(3):
                run(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(args.iters):
                run(i)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / args.iters * 1e3
            print(f"{args.model} {name:7s} tokens={M} pair={pair} split={split} stages={args.stages}: "
                  f"{us:7.1f} us  {N * K * 2 / us / 1e3:6.0f} GB/s", flush=True)
        assert int(status.item()) == 0
        del Ws


if __name__ == "__main__":
    main()
