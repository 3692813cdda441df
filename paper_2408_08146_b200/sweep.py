"""Kernel-level sweep on the 7B shapes: draft latency against K, verify latency against tree size,
context length and batch, each with its algorithmic bytes and the fraction of the HBM roofline.

    python -m paper_2408_08146_b200.sweep [--what draft,verify,medusa] [--reps 10] [--json out.json]

Run from the repository root (the seeded weight generator lives in `workloads/`).  Caches are
zero-filled (the timing does not depend on their contents); lengths are set directly.
The draft sweep runs whole iterations of an EAGLE-style head (D = 5 passes, top-10, 60-node tree,
context 1024) on top of a one-layer target and times the draft / expand_tree calls only.
The verify sweep times koala_verify on caller-supplied random trees.
The medusa sweep times the Medusa-style draft with the shared LM head and with a Linear per head.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import T13_EAGLE, T33_EAGLE, T7_EAGLE, T7_MEDUSA  # noqa: E402
from workloads.generate import WeightStore, medusa_static_tree, uniform_ints  # noqa: E402

from . import Koala  # noqa: E402

DEV = "cuda:0"
NOMINAL_GBS = 8000.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(path))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
    except Exception:
        return 6650.0, 1590.0, "fallback"


def layer_bytes(c):
    return (4 * c.H * c.H + 3 * c.H * c.F) * 2


def timed(fn, reps, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def random_tree(cfg, n, seed):
    """Random parents (parent < child), random tokens, as device arrays for koala_verify."""
    tok = uniform_ints(seed, "sweep.tok", cfg.B * n, 0, cfg.V).reshape(cfg.B, n)
    par = np.zeros((cfg.B, n), np.int32)
    r = uniform_ints(seed, "sweep.par", cfg.B * n, 0, 1 << 30).reshape(cfg.B, n)
    for b in range(cfg.B):
        par[b, 0] = -1
        for u in range(1, n):
            par[b, u] = max(0, u - 1 - int(r[b, u]) % min(u, 6))       # shallow-ish tree, depth grows slowly
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    return to(tok), to(par), to(np.full(cfg.B, n, np.int32)), n


def draft_sweep(store, reps, peak, base=T7_EAGLE, Ks=(1, 2, 3, 4)):
    rows = []
    S = 1024
    for K in Ks:
        cfg = base.with_(L=1, K=K, S_max=S + 256, B=1)
        eng = Koala(cfg, store.tensors)
        bufs = eng.buffers()
        eng.seq_len.fill_(S)
        bufs["n_pend"].fill_(3)
        forced = torch.full((cfg.B,), 3, dtype=torch.int32, device=DEV)
        stream = torch.cuda.current_stream()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * cfg.D + 1)]
        per_pass = np.zeros(cfg.D)
        total = 0.0
        n = 0
        for it in range(3 + reps):
            eng.seq_len.fill_(S)                      # keep the context length fixed across iterations
            for p in range(cfg.D):
                ev[2 * p].record(stream)
                eng.koala_draft(p)
                eng.koala_expand_tree(p)
                ev[2 * p + 1].record(stream)
            eng.koala_verify(None)
            eng.koala_accept(forced)
            torch.cuda.synchronize()
            if it >= 3:
                t = [ev[2 * p].elapsed_time(ev[2 * p + 1]) for p in range(cfg.D)]
                per_pass += np.asarray(t)
                total += ev[0].elapsed_time(ev[2 * cfg.D - 1])
                n += 1
        assert eng.device_status() == 0
        per_pass /= n
        total /= n
        # fc [H][2H] + K layers + LM head, plus the head's own KV context
        bytes_pass = 2 * cfg.H * cfg.H * 2 + K * layer_bytes(cfg) + cfg.V * cfg.H * 2 + K * S * cfg.H * 2 * 2
        gbs = cfg.D * bytes_pass / (total * 1e-3) / 1e9
        rows.append({"K": K, "context": S, "passes": cfg.D, "ms_per_pass": [round(float(x), 4) for x in per_pass],
                     "ms_per_iteration": round(total, 4), "bytes_per_pass": bytes_pass, "GBps": round(gbs, 1),
                     "frac_measured": round(gbs / peak, 3), "frac_8TBps": round(gbs / NOMINAL_GBS, 3)})
        print(f"draft  K={K}: {total:7.3f} ms / iteration of {cfg.D} passes "
              f"({' '.join('%.3f' % x for x in per_pass)}), {bytes_pass / 1e6:7.1f} MB/pass, {gbs:6.0f} GB/s = "
              f"{gbs / peak:.2f} of measured, {gbs / NOMINAL_GBS:.2f} of 8 TB/s", flush=True)
        eng.close()
        del eng
    return rows


def medusa_sweep(reps, peak):
    """Medusa-style draft (4 heads x K = 2 residual blocks, one pass): the shared LM head against a
    Linear of its own per head (Section 3.1's head as drawn), on a one-layer target."""
    rows = []
    for own in (False, True):
        cfg = T7_MEDUSA.with_(L=1, medusa_own_lm=own, S_max=768)
        store = WeightStore(cfg, DEV)
        eng = Koala(cfg, store.tensors, static_tree=medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk))
        eng.seq_len.fill_(512)
        bufs = eng.buffers()
        bufs["n_pend"].fill_(3)
        forced = torch.full((cfg.B,), 3, dtype=torch.int32, device=DEV)
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        total, n = 0.0, 0
        for it in range(3 + reps):
            eng.seq_len.fill_(512)
            e0.record(stream)
            eng.koala_draft(0)
            eng.koala_expand_tree(0)
            e1.record(stream)
            eng.koala_verify(None)
            eng.koala_accept(forced)
            torch.cuda.synchronize()
            if it >= 3:
                total += e0.elapsed_time(e1)
                n += 1
        assert eng.device_status() == 0
        ms = total / n
        nbytes = cfg.n_medusa_heads * cfg.K * cfg.H * cfg.H * 2 + (cfg.n_medusa_heads if own else 1) * cfg.V * cfg.H * 2
        gbs = nbytes / (ms * 1e-3) / 1e9
        rows.append({"own_linear": own, "ms": round(ms, 4), "bytes": nbytes, "GBps": round(gbs, 1),
                     "frac_measured": round(gbs / peak, 3)})
        print(f"medusa draft, {'a Linear per head' if own else 'shared LM head   '}: {ms:6.3f} ms, {nbytes / 1e6:7.1f} MB, "
              f"{gbs:6.0f} GB/s = {gbs / peak:.2f} of measured, {gbs / NOMINAL_GBS:.2f} of 8 TB/s", flush=True)
        eng.close()
        del eng, store
        torch.cuda.empty_cache()
    return rows


def verify_sweep(store, reps, peak, tflops, base=T7_EAGLE, grid=None):
    rows = []
    if grid is None:
        grid = [(n, s, 1) for n in (16, 32, 64, 128) for s in (128, 512, 2048, 4096)]
        grid += [(64, 512, b) for b in (2, 4, 8)] + [(64, 2048, b) for b in (2, 4, 8)]
    base = base.with_(K=1)
    wbytes = base.L * layer_bytes(base) + base.V * base.H * 2
    for n, s, b in grid:
        cfg = base.with_(N=n, B=b, S_max=((s + n + 127) // 128) * 128, D=min(base.D, max(1, n - 1)))
        eng = Koala(cfg, store.tensors)
        eng.seq_len.fill_(s)
        tree = random_tree(cfg, n, 77)
        ms = timed(lambda: eng.koala_verify(tree), reps)
        assert eng.device_status() == 0
        kv = cfg.L * b * s * cfg.H * 2 * 2
        gbs = (wbytes + kv) / (ms * 1e-3) / 1e9
        flops = 2.0 * (wbytes / 2) * n * b
        t_hbm = (wbytes + kv) / (peak * 1e9) * 1e3
        t_tc = flops / (tflops * 1e12) * 1e3
        rows.append({"tree": n, "context": s, "batch": b, "rows": n * b, "ms": round(ms, 4), "bytes": wbytes + kv,
                     "GBps": round(gbs, 1), "frac_measured": round(gbs / peak, 3),
                     "frac_8TBps": round(gbs / NOMINAL_GBS, 3), "ideal_ms_hbm": round(t_hbm, 3),
                     "ideal_ms_tensor": round(t_tc, 3), "bound": "hbm" if t_hbm >= t_tc else "tensor"})
        print(f"verify N={n:3d} S={s:4d} B={b}: {ms:7.3f} ms, {(wbytes + kv) / 1e9:6.2f} GB, {gbs:6.0f} GB/s = "
              f"{gbs / peak:.2f} of measured, {gbs / NOMINAL_GBS:.2f} of 8 TB/s  (ideal {t_hbm:.2f} ms hbm / "
              f"{t_tc:.2f} ms tensor)", flush=True)
        eng.close()
        del eng
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--what", default="draft,verify")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--json", default="")
    ap.add_argument("--model", default="7b", choices=["7b", "13b", "33b"],
                    help="13b: the 13B shape at batch 1 and 4 (tree 64, context 2048); "
                         "33b: the 33B shape (65 GB of weights): draft K = 1..8, verify at three points")
    args = ap.parse_args()
    peak, tflops, src = measured_peak()
    print(f"HBM peak {peak:.0f} GB/s ({src}); nominal {NOMINAL_GBS:.0f} GB/s")
    out = {"peak_GBps": peak, "peak_source": src}
    if "medusa" in args.what:
        out["medusa"] = medusa_sweep(args.reps, peak)
    if args.model == "13b":
        store = WeightStore(T13_EAGLE.with_(K=2), DEV)
        if "draft" in args.what:
            out["draft"] = draft_sweep(store, args.reps, peak, T13_EAGLE, (1, 2))
        if "verify" in args.what:
            out["verify"] = verify_sweep(store, args.reps, peak, tflops, T13_EAGLE,
                                         [(64, 512, 1), (64, 2048, 1), (64, 2048, 4)])
        if args.json:
            json.dump(out, open(args.json, "w"), indent=1)
        return
    if args.model == "33b":
        store = WeightStore(T33_EAGLE.with_(K=8), DEV)
        if "draft" in args.what:
            out["draft"] = draft_sweep(store, args.reps, peak, T33_EAGLE, (1, 2, 4, 6, 8))
        if "verify" in args.what:
            out["verify"] = verify_sweep(store, args.reps, peak, tflops, T33_EAGLE, [(16, 512, 1), (60, 512, 1), (60, 2048, 1)])
        if args.json:
            json.dump(out, open(args.json, "w"), indent=1)
        return
    store = WeightStore(T7_EAGLE.with_(K=4), DEV) if ("draft" in args.what or "verify" in args.what) else None
    if "draft" in args.what:
        out["draft"] = draft_sweep(store, args.reps, peak)
    if "verify" in args.what:
        out["verify"] = verify_sweep(store, args.reps, peak, tflops)
    if args.json:
        json.dump(out, open(args.json, "w"), indent=1)


if __name__ == "__main__":
    main()
