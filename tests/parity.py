"""Comparison rules between the CUDA library and the oracle.

Floating point: an element passes if |gpu - ref| <= atol or |gpu - ref| <= rtol * |ref|
(bf16 configurations: atol 3e-2, rtol 2e-2; the fp32 configuration: atol 1e-4, rtol 1e-4).
Integers (token ids, tree indices, accepted lengths) must be equal, except where the decision
rests on a comparison whose two oracle-side operands differ by less than 1e-2 (near tie).
"""
import numpy as np

TIE = 1e-2
TOL = {0: (1e-4, 1e-4), 1: (3e-2, 2e-2)}   # dtype -> (atol, rtol)


def assert_close(gpu, ref, dtype, what, atol=None, rtol=None):
    a, r = TOL[dtype]
    atol = a if atol is None else atol
    rtol = r if rtol is None else rtol
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, f"{what}: shape {gpu.shape} vs {ref.shape}"
    assert np.isfinite(gpu).all(), f"{what}: non-finite values from the GPU"
    err = np.abs(gpu - ref)
    bad = ~((err <= atol) | (err <= rtol * np.abs(ref)))
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} elements out of tolerance; "
                           f"max abs err {err.max():.3e} (ref scale {np.abs(ref).max():.3e})")
    if err.size:
        print(f"[parity] {what}: max abs err {err.max():.3e}, rms err {np.sqrt(np.mean(err ** 2)):.3e}, "
              f"ref rms {np.sqrt(np.mean(ref ** 2)):.3e}")
    return float(err.max()) if err.size else 0.0


def check_argmax(gpu_idx, ref_logits, what):
    """Every row's index equals the oracle's arg-max unless the oracle's gap to it is < TIE."""
    excused = 0
    for r, g in enumerate(np.asarray(gpu_idx).reshape(-1)):
        row = ref_logits[r]
        best = int(np.argmax(row))
        if int(g) != best:
            assert row[best] - row[int(g)] < TIE, f"{what}: row {r} picked {g}, oracle {best}"
            excused += 1
    return excused


def check_topk(gpu_tok, ref_logits_row, k, what):
    """Position-wise: a differing token is excused only if its oracle logit is within TIE of the
    oracle's choice at that position."""
    order = np.lexsort((np.arange(ref_logits_row.shape[0]), -ref_logits_row))[:k]
    excused = 0
    for j in range(k):
        g = int(gpu_tok[j])
        if g != int(order[j]):
            assert abs(ref_logits_row[order[j]] - ref_logits_row[g]) < TIE, \
                f"{what}: rank {j} picked {g}, oracle {order[j]}"
            excused += 1
    return excused
