"""Closed-form pins of the oracle's elementary operations."""
import itertools

import numpy as np

from oracle.koala_oracle import (argmax_first, log_softmax, masked_softmax, rmsnorm, rope,
                                 round_to_bf16, silu, top_k)

RNG = np.random.default_rng(11)


def test_rope_hand_example_and_invariants():
    # dh = 2: a single pair rotated by pos * base**0 = pos radians
    x = np.asarray([[[1.0, 0.0]]])
    y = rope(x, np.asarray([1]), 10000.0)
    assert np.allclose(y[0, 0], [np.cos(1.0), np.sin(1.0)])
    # dh = 4: pairs (0, 2) and (1, 3); second pair turns by pos * base**(-1/2)
    x = np.asarray([[[1.0, 2.0, 3.0, 4.0]]])
    y = rope(x, np.asarray([3]), 100.0)[0, 0]
    a, b = 3.0, 3.0 * 100.0 ** -0.5
    assert np.allclose(y, [np.cos(a) - 3 * np.sin(a), 2 * np.cos(b) - 4 * np.sin(b),
                           3 * np.cos(a) + np.sin(a), 4 * np.cos(b) + 2 * np.sin(b)])
    q = RNG.standard_normal((5, 3, 16))
    k = RNG.standard_normal((5, 3, 16))
    pos = np.asarray([0, 1, 7, 100, 1000])
    rq = rope(q, pos, 10000.0)
    assert np.allclose(rq[0], q[0])                                         # position 0: identity
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1))   # a rotation
    # <rope(q, m), rope(k, n)> depends on m - n only
    d1 = np.sum(rope(q[:1], np.asarray([12]), 1e4) * rope(k[:1], np.asarray([5]), 1e4))
    d2 = np.sum(rope(q[:1], np.asarray([107]), 1e4) * rope(k[:1], np.asarray([100]), 1e4))
    assert abs(d1 - d2) < 1e-9


def test_rmsnorm_closed_form():
    x = np.asarray([[3.0, 4.0]])
    g = np.asarray([2.0, 0.5])
    # mean square = 12.5
    assert np.allclose(rmsnorm(x, g, 0.0), [[2 * 3 / np.sqrt(12.5), 0.5 * 4 / np.sqrt(12.5)]])
    assert np.allclose(rmsnorm(x, g, 3.5), [[2 * 3 / 4.0, 0.5 * 4 / 4.0]])
    y = rmsnorm(RNG.standard_normal((4, 64)), np.ones(64), 0.0)
    assert np.allclose(np.mean(y * y, axis=-1), 1.0)


def test_silu_and_softmax():
    assert silu(np.asarray(0.0)) == 0.0
    assert np.allclose(silu(np.asarray([1.0, -1.0])), [1 / (1 + np.exp(-1)), -1 / (1 + np.exp(1))])
    s = RNG.standard_normal((3, 6)) * 5
    vis = np.asarray([[1, 1, 0, 0, 1, 0], [1, 0, 0, 0, 0, 0], [1, 1, 1, 1, 1, 1]], dtype=bool)
    p = masked_softmax(s, vis)
    assert np.allclose(p.sum(-1), 1.0) and np.all(p[~vis] == 0.0)
    assert np.allclose(p[1], [1, 0, 0, 0, 0, 0])
    assert np.allclose(p[2], np.exp(s[2]) / np.exp(s[2]).sum())
    z = np.asarray([[0.0, np.log(3.0)]])
    assert np.allclose(log_softmax(z), [[np.log(0.25), np.log(0.75)]])
    big = np.asarray([[1000.0, 1000.0]])
    assert np.allclose(log_softmax(big), np.log(0.5))                       # max-subtracted


def test_top_k_against_brute_force_with_ties():
    for trial in range(50):
        v = RNG.integers(0, 6, size=12).astype(np.float64)                  # many ties
        k = int(RNG.integers(1, 12))
        got = list(top_k(v, k))
        # brute force: repeatedly take the first maximum
        rest, want = list(range(12)), []
        for _ in range(k):
            best = max(v[i] for i in rest)
            i = min(i for i in rest if v[i] == best)
            want.append(i)
            rest.remove(i)
        assert got == want
    assert argmax_first(np.asarray([1.0, 5.0, 5.0, 2.0])) == 1


def test_bf16_storage_rounding_matches_the_library_conversion():
    import torch
    x = (RNG.standard_normal(200000) * np.exp(RNG.uniform(-20, 20, 200000))).astype(np.float32)
    # exact ties (low 16 bits = 0x8000) round to even
    ties = (RNG.integers(0x3F00, 0x4100, 1000).astype(np.uint32) << np.uint32(16)) | np.uint32(0x8000)
    x = np.concatenate([x, ties.view(np.float32), np.asarray([0.0, -0.0, 1.0, -1.0, 3.140625], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = round_to_bf16(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert round_to_bf16(np.asarray([1.00390625], np.float32))[0] == 1.0          # 1 + 2^-8: tie -> even
    assert round_to_bf16(np.asarray([1.01171875], np.float32))[0] == 1.015625     # 1 + 3*2^-8: tie -> even
