"""Pins of acceptance, compaction and the whole loop: losslessness against greedy decoding."""
import numpy as np
import pytest

from oracle.koala_oracle import KoalaOracle
from tests.helpers import HostWeights
from workloads import TINY_EAGLE, TINY_MEDUSA
from workloads.generate import WeightStore, medusa_static_tree, prompts

CFG = TINY_EAGLE.with_(S_max=160)


@pytest.fixture(scope="module")
def hw():
    return HostWeights(WeightStore(CFG))


@pytest.fixture(scope="module")
def ar_stream(hw):
    o = KoalaOracle(CFG, hw)
    o.prefill(prompts(CFG), 64)
    first_root = o.root_tok[0]
    return first_root, o.ar_greedy(48)[0]


def _planted_tree(rng, truth, m, n_nodes, V):
    """Random tree whose one branch spells truth[0:m]; every other node carries a wrong token.

    truth[i] is the greedy token that follows the path's i-th node.  Returns (tok, parent)
    without the root token (filled by the caller).
    """
    parent, depth_truth = [-1], {0: 0}          # node -> how many truth tokens its path spells
    tok = [None]
    on_path = 0
    for _ in range(m):                           # the planted branch
        parent.append(on_path)
        tok.append(int(truth[depth_truth[on_path]]))
        depth_truth[len(parent) - 1] = depth_truth[on_path] + 1
        on_path = len(parent) - 1
    while len(parent) < n_nodes:                 # junk nodes anywhere
        par = int(rng.integers(0, len(parent)))
        forbidden = int(truth[depth_truth[par]]) if par in depth_truth else -1
        sib = {tok[v] for v in range(1, len(parent)) if parent[v] == par}
        t = int(rng.integers(0, V))
        while t == forbidden or t in sib:
            t = int(rng.integers(0, V))
        parent.append(par)
        tok.append(t)
    # renumber so parents precede children in (level, parent, arrival) order
    order = sorted(range(len(parent)), key=lambda u: (_lvl(parent, u), u))
    new_of = {u: i for i, u in enumerate(order)}
    tok2 = [tok[u] for u in order]
    par2 = [-1 if parent[u] < 0 else new_of[parent[u]] for u in order]
    return tok2, par2


def _lvl(parent, u):
    d = 0
    while parent[u] >= 0:
        u = parent[u]
        d += 1
    return d


def test_planted_paths_and_losslessness(hw, ar_stream):
    """Greedy speculative decoding emits exactly the greedy autoregressive stream, and a tree
    that contains the true continuation for m tokens is accepted for exactly m + 1 tokens."""
    first_root, truth = ar_stream
    rng = np.random.default_rng(5)
    o = KoalaOracle(CFG, hw)
    o.prefill(prompts(CFG), 16)
    assert o.root_tok[0] == first_root
    emitted = []
    while len(emitted) < 36:
        m = int(rng.integers(0, 5))
        tok, par = _planted_tree(rng, truth[len(emitted):], m, int(rng.integers(m + 1, 16)), CFG.V)
        tok[0] = o.root_tok[0]
        s_before = o.seq_len[0]
        o.verify([(np.asarray(tok), np.asarray(par))])
        toks, lens = o.accept()
        assert lens[0] == m + 1 and len(toks[0]) == m + 1
        assert o.seq_len[0] == s_before + lens[0]
        emitted += toks[0]
    assert emitted == truth[:len(emitted)]


@pytest.mark.parametrize("cfg", [TINY_EAGLE, TINY_MEDUSA], ids=["eagle", "medusa"])
def test_real_heads_are_lossless(cfg):
    cfg = cfg.with_(S_max=160)
    hw = HostWeights(WeightStore(cfg))
    st = medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk) if cfg.head_kind else None
    o = KoalaOracle(cfg, hw, static_tree=st)
    o.prefill(prompts(cfg), 16)
    spec, total = [], 0
    for _ in range(8):
        toks, lens = o.step()
        assert 1 <= lens[0] <= cfg.D + 1
        spec += toks[0]
        total += lens[0]
    assert total == len(spec) == o.seq_len[0] - cfg.prompt_len
    ref = KoalaOracle(cfg, hw, static_tree=st)
    ref.prefill(prompts(cfg), 64)
    assert ref.ar_greedy(len(spec))[0] == spec


def test_cache_after_acceptance_equals_direct_prefill(hw, ar_stream):
    first_root, truth = ar_stream
    rng = np.random.default_rng(9)
    o = KoalaOracle(CFG, hw)
    prompt = prompts(CFG)[0]
    o.prefill([prompt], 64)
    tok, par = _planted_tree(rng, truth, 3, 12, CFG.V)
    tok[0] = o.root_tok[0]
    o.verify([(np.asarray(tok), np.asarray(par))])
    toks, lens = o.accept()
    assert lens == [4] and toks[0] == truth[:4]
    direct = KoalaOracle(CFG, hw)
    full = list(prompt) + [first_root] + truth[:3]
    direct.prefill([full], len(full))
    assert direct.seq_len == o.seq_len == [68]
    for l in range(CFG.L):
        assert np.max(np.abs(direct.target_k[l][0][:68] - o.target_k[l][0][:68])) < 1e-10
        assert np.max(np.abs(direct.target_v[l][0][:68] - o.target_v[l][0][:68])) < 1e-10
    # hidden rows kept for the next draft pass are those of the accepted positions
    assert np.max(np.abs(direct.pend_hid[0][-4:] - o.pend_hid[0])) < 1e-9
    assert o.pend_tok[0] == truth[:3] and o.root_tok[0] == truth[3]


def test_forced_length_rule_and_duplicate_siblings(hw):
    o = KoalaOracle(CFG, hw)
    o.prefill(prompts(CFG), 64)
    root = o.root_tok[0]
    #  0 -> {1, 2}; 1 -> {3}; 2 -> {4, 5}; 3 -> {6}
    parent = np.asarray([-1, 0, 0, 1, 2, 2, 3])

    def run(tok, tgt, forced):
        o.tree_tok[0], o.tree_parent[0] = np.asarray(tok), parent
        o.verify_tgt[0] = np.asarray(tgt)
        o.verify_hid[0] = np.zeros((7, CFG.H))
        s = o.seq_len[0]
        toks, lens = o.accept(forced)
        o.seq_len[0] = s
        return toks[0], lens[0]

    tok = [root, 10, 20, 30, 40, 50, 60]
    # natural: target says 20 after the root, 50 after node 2, 99 after node 5
    assert run(tok, [20, 0, 50, 0, 0, 99, 0], None) == ([20, 50, 99], 3)
    # no match at all: only the bonus token
    assert run(tok, [77, 0, 0, 0, 0, 0, 0], None) == ([77], 1)
    # forced 4, nothing matches: lowest-numbered children 1, 3, 6
    assert run(tok, [77, 78, 0, 79, 0, 0, 80], [4]) == ([10, 30, 60, 80], 4)
    # forced 6 stops at the leaf (4 nodes on the deepest left path)
    assert run(tok, [77, 78, 0, 79, 0, 0, 80], [6]) == ([10, 30, 60, 80], 4)
    # forced 2 while the target matches a deeper path: stops at 2 nodes, bonus from node 2
    assert run(tok, [20, 0, 50, 0, 0, 99, 0], [2]) == ([20, 50], 2)
    # forced prefers a matching child over the lowest-numbered one
    assert run(tok, [20, 0, 0, 0, 11, 0, 0], [3]) == ([20, 40, 11], 3)
    # forced 1: the root alone
    assert run(tok, [20, 0, 50, 0, 0, 99, 0], [1]) == ([20], 1)
    # duplicate sibling tokens: the lower-numbered child wins
    dup = [root, 20, 20, 30, 40, 50, 60]
    assert run(dup, [20, 5, 6, 0, 0, 0, 0], None) == ([20, 5], 2)


def test_position_wise_acceptance_counts_on_planted_chains(hw, ar_stream):
    """n-alpha (Section 4.1, metrics: accuracy of the n-th drafted token, chain drafts): a chain of
    depth d whose first m tokens are the true continuation offers positions 1 .. min(m + 1, d)
    and hits positions 1 .. m.  The expected counts are tallied here from (m, d) alone."""
    first_root, truth = ar_stream
    rng = np.random.default_rng(11)
    o = KoalaOracle(CFG, hw)
    o.prefill(prompts(CFG), 16)
    o.reset_alpha()
    hits, trials = [0] * CFG.N, [0] * CFG.N
    emitted = 0
    for _ in range(14):
        d = int(rng.integers(1, 5))
        m = int(rng.integers(0, d + 1))
        tok = [o.root_tok[0]]
        for i in range(d):
            t = int(truth[emitted + i])
            tok.append(t if i < m else (t + 1 + int(rng.integers(0, CFG.V - 1))) % CFG.V)
        par = list(range(-1, d))
        o.verify([(np.asarray(tok), np.asarray(par))])
        _, lens = o.accept()
        assert lens[0] == m + 1
        emitted += lens[0]
        for n in range(1, d + 1):
            if n <= m + 1:
                trials[n - 1] += 1
            if n <= m:
                hits[n - 1] += 1
    assert o.alpha_hits == hits and o.alpha_trials == trials
    assert all(h <= t for h, t in zip(hits, trials)) and trials[0] == 14
    # a bushy tree counts the walked path only: the same tally with junk siblings around
    o.reset_alpha()
    tok, par = _planted_tree(rng, truth[emitted:], 2, 12, CFG.V)
    tok[0] = o.root_tok[0]
    o.verify([(np.asarray(tok), np.asarray(par))])
    _, lens = o.accept()
    assert lens[0] == 3 and o.alpha_hits[:3] == [1, 1, 0]
    assert o.alpha_trials[:2] == [1, 1] and o.alpha_trials[2] in (0, 1)     # 1 iff the path's end has a (wrong) child
