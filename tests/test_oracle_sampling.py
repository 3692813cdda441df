"""Pins of the speculative-sampling acceptance (Section 2.2, the paragraph after Eq. 3) against
what the method guarantees: the emitted tokens are distributed as if the target had sampled them."""
import numpy as np

from oracle.koala_oracle import KoalaOracle, log_softmax, sample_index, speculative_sampling_step
from tests.helpers import HostWeights
from workloads import TINY_EAGLE
from workloads.generate import WeightStore, prompts


def test_inverse_cdf_draw_matches_a_hand_walk():
    w = np.asarray([0.0, 0.2, 0.0, 0.5, 0.3, 0.0])
    # cumulative 0, .2, .2, .7, 1.0, 1.0 -> boundaries at u = 0.2 and 0.7
    assert [sample_index(w, u) for u in (0.0, 0.1999, 0.2, 0.6999, 0.7, 0.9999)] == [1, 1, 3, 3, 4, 4]
    assert sample_index(np.asarray([0.0, 0.0, 2.0, 0.0]), 0.999999) == 2        # unnormalised weights
    rng = np.random.default_rng(0)
    w = rng.random(1000)
    draws = np.asarray([sample_index(w, u) for u in rng.random(20000)])
    freq = np.bincount(draws, minlength=1000) / 20000
    assert np.abs(freq - w / w.sum()).max() < 5 * np.sqrt((w / w.sum()).max() / 20000)


def test_identical_distributions_accept_everything_and_disjoint_ones_nothing():
    rng = np.random.default_rng(1)
    q = rng.random((4, 7)); q /= q.sum(axis=1, keepdims=True)
    drafted = [int(np.argmax(q[i])) for i in range(3)]
    for u in (0.0, 0.5, 0.999999):
        a, bonus = speculative_sampling_step(q[:3], q, drafted, [u] * 3, 0.3)
        assert a == 3 and bonus == sample_index(q[3], 0.3)
    # the draft puts all its mass where the target has none: rejected at once, and the residual
    # max(0, q - d) is q itself
    d0 = np.zeros(7); d0[2] = 1.0
    q0 = q[0].copy(); q0[2] = 0.0; q0 /= q0.sum()
    a, bonus = speculative_sampling_step([d0], [q0, q[1]], [2], [0.0], 0.77)
    assert a == 0 and bonus == sample_index(q0, 0.77)


def test_emitted_tokens_follow_the_target_distribution():
    """Monte Carlo over the uniforms with fixed d_i, q_i (V = 6, t = 2): the first emitted token is
    distributed as q_1 and, when a second one is emitted, it is distributed as q_2 - whatever the
    draft distributions are.  300 000 trials, bounds at five standard deviations."""
    rng = np.random.default_rng(2)
    V, t, M = 6, 2, 300_000
    d = rng.random((t, V)) ** 3; d /= d.sum(axis=1, keepdims=True)
    q = rng.random((t + 1, V)) ** 2; q /= q.sum(axis=1, keepdims=True)
    first = np.zeros(V); second = np.zeros(V); n_second = 0; accepted = np.zeros(t + 1)
    U = rng.random((M, 2 * t + 1))
    for m in range(M):
        drafted = [sample_index(d[i], U[m, i]) for i in range(t)]
        a, bonus = speculative_sampling_step(d, q, drafted, U[m, t:2 * t], U[m, 2 * t])
        out = drafted[:a] + [bonus]
        first[out[0]] += 1
        accepted[a] += 1
        if len(out) >= 2:
            second[out[1]] += 1
            n_second += 1
    assert np.abs(first / M - q[0]).max() < 5 * np.sqrt(0.25 / M)
    assert np.abs(second / n_second - q[1]).max() < 5 * np.sqrt(0.25 / n_second)
    # acceptance probability of the first token: sum_x min(d_1(x), q_1(x))
    p1 = np.minimum(d[0], q[0]).sum()
    assert abs((1 - accepted[0] / M) - p1) < 5 * np.sqrt(0.25 / M)


def test_sampled_chain_through_the_whole_oracle():
    """Chain drafts of an EAGLE-style head with sampled tokens: the kept draft distributions are
    the softmax of the head's logits, the chain is the sampled tokens, and accept_sampled agrees
    with the stand-alone step on the oracle's own q and d."""
    cfg = TINY_EAGLE.with_(topk=1, D=3, N=4, S_max=160)
    o = KoalaOracle(cfg, HostWeights(WeightStore(cfg)))
    o.prefill(prompts(cfg), 16)
    rng = np.random.default_rng(3)
    for it in range(5):
        U = rng.random(cfg.D + cfg.D + 1)
        for p in range(cfg.D):
            o.draft(p)
            logits = o.draft_logits[0][0].copy()
            o.expand_tree(p, u_draft=[U[p]])
            np.testing.assert_allclose(o.chain_d[0][p], np.exp(log_softmax(logits)), rtol=0, atol=1e-15)
        assert list(o.tree_parent[0]) == [-1, 0, 1, 2]
        assert [int(t) for t in o.tree_tok[0][1:]] == [sample_index(o.chain_d[0][p], U[p]) for p in range(cfg.D)]
        o.verify()
        q = np.exp(log_softmax(o.verify_logits[0]))
        a_ref, bonus_ref = speculative_sampling_step([o.chain_d[0][p] for p in range(cfg.D)], q,
                                                     [int(t) for t in o.tree_tok[0][1:]], U[cfg.D:2 * cfg.D], U[-1])
        s_before = o.seq_len[0]
        toks, lens = o.accept_sampled([U[cfg.D:2 * cfg.D]], [U[-1]])
        assert lens[0] == a_ref + 1 and toks[0][-1] == bonus_ref and o.root_tok[0] == bonus_ref
        assert o.seq_len[0] == s_before + lens[0]
