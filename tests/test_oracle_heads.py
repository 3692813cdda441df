"""Pins of the draft heads (Section 3.1 structures) and of the tree expansion."""
import numpy as np
import pytest

from oracle.koala_oracle import (KoalaOracle, ancestor_matrix, log_softmax, rmsnorm, top_k,
                                 tree_levels)
from tests.helpers import HostWeights
from workloads import TINY_EAGLE, TINY_MEDUSA
from workloads.generate import WeightStore, medusa_static_tree, prompts

ECFG = TINY_EAGLE.with_(S_max=128)
MCFG = TINY_MEDUSA.with_(S_max=128)


def _medusa(cfg, hw):
    st = medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk)
    o = KoalaOracle(cfg, hw, static_tree=st)
    o.prefill(prompts(cfg), 32)
    return o


# ------------------------------------------------------------------------------- Medusa-style
def test_medusa_without_blocks_reproduces_the_target_logits():
    """K = 0: every head is the bare LM head on the target's last hidden state."""
    cfg = MCFG.with_(K=0)
    o = _medusa(cfg, HostWeights(WeightStore(cfg)))
    last_logits = o.verify_logits[0][-1]
    o.draft(0)
    for i in range(cfg.n_medusa_heads):
        assert np.max(np.abs(o.draft_logits[0][i] - last_logits)) < 1e-12
    assert int(np.argmax(o.draft_logits[0][0])) == o.root_tok[0]


def test_medusa_zero_block_is_identity_and_scalar_block_closed_form():
    hw = HostWeights(WeightStore(MCFG))
    H = MCFG.H
    for i in range(MCFG.n_medusa_heads):
        for j in range(MCFG.K):
            hw.override(f"medusa.{i}.{j}.w", np.zeros((H, H)))
            hw.override(f"medusa.{i}.{j}.b", np.zeros(H))
    o = _medusa(MCFG, hw)
    o.draft(0)
    assert np.max(np.abs(o.draft_feat[0] - o.pend_hid[0][-1][None, :])) == 0.0     # SiLU(0) = 0
    # W = I, b = 0, K = 1, input of ones: 1 + 1/(1 + e^-1) = 1.7310585786300048
    cfg1 = MCFG.with_(K=1)
    hw1 = HostWeights(WeightStore(cfg1))
    for i in range(cfg1.n_medusa_heads):
        hw1.override(f"medusa.{i}.0.w", np.eye(H)).override(f"medusa.{i}.0.b", np.zeros(H))
    o1 = KoalaOracle(cfg1, hw1)
    _, feats = o1.medusa_draft(np.ones(H))
    assert np.allclose(feats, 1.7310585786300048, atol=1e-15)
    # bias enters inside the SiLU: W = 0, b = 2 -> x + 2/(1+e^-2)
    for i in range(cfg1.n_medusa_heads):
        hw1.override(f"medusa.{i}.0.w", np.zeros((H, H))).override(f"medusa.{i}.0.b", np.full(H, 2.0))
    _, feats = o1.medusa_draft(np.full(H, 0.5))
    assert np.allclose(feats, 0.5 + 2.0 / (1.0 + np.exp(-2.0)), atol=1e-15)


def test_medusa_k_blocks_compose_and_heads_are_independent():
    hw = HostWeights(WeightStore(MCFG))
    o = KoalaOracle(MCFG, hw)
    h = np.random.default_rng(0).standard_normal(MCFG.H)
    _, feats2 = o.medusa_draft(h)
    cfg1 = MCFG.with_(K=1)
    for i in range(MCFG.n_medusa_heads):
        first = HostWeights(WeightStore(MCFG))
        o_a = KoalaOracle(cfg1, first)                                   # block (i, 0)
        x = o_a.medusa_draft(h)[1][i]
        second = HostWeights(WeightStore(MCFG))
        second.override(f"medusa.{i}.0.w", hw(f"medusa.{i}.1.w")).override(
            f"medusa.{i}.0.b", hw(f"medusa.{i}.1.b"))
        x = KoalaOracle(cfg1, second).medusa_draft(x)[1][i]             # then block (i, 1)
        assert np.max(np.abs(x - feats2[i])) < 1e-12
    assert np.max(np.abs(feats2[0] - feats2[1])) > 1e-3                  # heads differ


def test_medusa_expansion_fills_the_static_tree_by_rank():
    o = _medusa(MCFG, HostWeights(WeightStore(MCFG)))
    o.draft(0)
    o.expand_tree(0)
    parent, level, rank = o.static_tree
    tok = o.tree_tok[0]
    assert tok[0] == o.root_tok[0] and list(o.tree_parent[0]) == list(parent)
    for u in range(1, len(parent)):
        row = o.draft_logits[0][level[u] - 1]
        # brute force: the token with exactly rank[u] strictly better entries
        better = np.sum((row > row[tok[u]]) | ((row == row[tok[u]]) & (np.arange(len(row)) < tok[u])))
        assert better == rank[u]


# -------------------------------------------------------------------------------- EAGLE-style
def _eagle(cfg, hw, chunk=16):
    o = KoalaOracle(cfg, hw)
    o.prefill(prompts(cfg), chunk)
    return o


def test_eagle_fc_reads_hidden_then_embedding():
    """With K = 0 the head is LM(W_fc [h ; e] + b): selector matrices expose the operand order."""
    cfg = ECFG.with_(K=0)
    H = cfg.H
    hw = HostWeights(WeightStore(cfg))
    hw.override("fc_b", np.zeros(H))
    hw.override("fc_w", np.concatenate([np.eye(H), np.zeros((H, H))], axis=1))      # picks h
    o = _eagle(cfg, hw)
    last_logits = o.verify_logits[0][-1]
    o.draft(0)
    assert np.max(np.abs(o.draft_logits[0][0] - last_logits)) < 1e-12               # LM(h_{S-1})
    assert int(np.argmax(o.draft_logits[0][0])) == o.root_tok[0]
    hw.override("fc_w", np.concatenate([np.zeros((H, H)), np.eye(H)], axis=1))      # picks E[x_S]
    o = _eagle(cfg, hw)
    o.draft(0)
    want = hw("embed")[o.root_tok[0]] @ hw("lm_head").T
    assert np.max(np.abs(o.draft_logits[0][0] - want)) < 1e-12
    hw.override("fc_w", np.zeros((H, 2 * H))).override("fc_b", np.arange(H) / H)    # bias alone
    o = _eagle(cfg, hw)
    o.draft(0)
    assert np.max(np.abs(o.draft_logits[0][0] - (np.arange(H) / H) @ hw("lm_head").T)) < 1e-12


def test_eagle_layer_stack_is_the_target_layer_applied_k_times():
    """Head layers := target layers, fc := embedding selector: the head's cache and feature
    equal the target stack run on the tokens shifted by one position."""
    cfg = ECFG.with_(K=ECFG.L)
    H = cfg.H
    hw = HostWeights(WeightStore(cfg))
    hw.override("fc_b", np.zeros(H))
    hw.override("fc_w", np.concatenate([np.zeros((H, H)), np.eye(H)], axis=1))
    for j in range(cfg.K):
        for t in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
            hw.override(f"draft.{j}.{t}", hw(f"layers.{j}.{t}"))
    prompt = prompts(cfg)[0][:24]
    o = KoalaOracle(cfg, hw)
    o.prefill([prompt], 8)
    o.draft(0)                                    # completes the head's cache to length S = 24
    shifted = list(prompt[1:]) + [o.root_tok[0]]
    ref = KoalaOracle(cfg, hw)
    logits, hid = ref.target_forward(0, np.asarray(shifted), np.arange(-1, 23))
    for j in range(cfg.K):
        assert np.max(np.abs(o.draft_k[j][0][:24] - ref.target_k[j][0][:24])) < 1e-10
        assert np.max(np.abs(o.draft_v[j][0][:24] - ref.target_v[j][0][:24])) < 1e-10
    # no norm between the last head layer and the LM head: applying the final norm afterwards
    # must give the target's normalised hidden state
    assert np.max(np.abs(rmsnorm(o.draft_feat[0][0], hw("final_norm"), cfg.rms_eps) - hid[-1])) < 1e-9


def test_eagle_tree_drafting_equals_chain_drafting_of_every_path():
    """A frontier node's predicted feature equals running the head along its root path as a
    chain: (parent's predicted feature, own token) at consecutive positions."""
    cfg = ECFG.with_(D=4, topk=3, N=20)
    hw = HostWeights(WeightStore(cfg))
    o = _eagle(cfg, hw)
    S = o.seq_len[0]
    feats, fronts = [], []
    for p in range(cfg.D):
        o.draft(p)
        feats.append(o.draft_feat[0].copy())
        fronts.append(list(o.frontier[0]))          # frontier that pass p just processed
        o.expand_tree(p)
    pool = o.pool[0]
    checked = 0
    for p in range(1, cfg.D):
        for i, cid in enumerate(fronts[p]):
            path = []
            a = cid
            while a != -1:
                path.append(a)
                a = pool[a]["parent"]
            path.reverse()
            assert len(path) == p
            ch = _eagle(cfg, hw)                   # fresh state, same context
            ch.draft(0)
            f = ch.draft_feat[0][0]
            for d, a in enumerate(path):
                n = d + 1
                vis = np.ones((1, S + n), dtype=bool)
                f_hat, _ = ch.eagle_forward(0, f[None, :], np.asarray([pool[a]["tok"]]),
                                            np.asarray([S + d]), np.asarray([S + d]), vis)
                f = f_hat[0]
            assert np.max(np.abs(f - feats[p][i])) < 1e-9
            checked += 1
    assert checked == (cfg.D - 1) * cfg.topk


def _check_tree_invariants(o, cfg):
    tok, parent, score = o.tree_tok[0], o.tree_parent[0], o.tree_score[0]
    n = len(tok)
    pool = o.pool[0]
    assert n == 1 + min(cfg.N - 1, len(pool))
    level = tree_levels(parent)
    key = [(level[u], parent[u]) for u in range(n)]
    assert key == sorted(key)                                      # (level, parent) order
    for u in range(1, n):
        assert score[u] <= score[parent[u]]                        # log-probs are <= 0
        sib = [v for v in range(1, n) if parent[v] == parent[u]]
        assert len({int(tok[v]) for v in sib}) == len(sib)
    # kept = the N-1 best scores of the pool (numpy sort as the independent routine)
    all_scores = np.sort(np.asarray([e["score"] for e in pool]))[::-1]
    kept_scores = np.sort(np.asarray(score[1:]))[::-1]
    assert np.array_equal(kept_scores, all_scores[: n - 1])
    return level


def test_dynamic_expansion_scores_frontier_and_selection():
    cfg = ECFG                                              # depth 4, top-2, 15 nodes
    o = _eagle(cfg, HostWeights(WeightStore(cfg)))
    logps, fronts = [], []
    for p in range(cfg.D):
        o.draft(p)
        logps.append(log_softmax(o.draft_logits[0]))
        fronts.append(list(o.frontier[0]))
        o.expand_tree(p)
        if 0 < p < cfg.D - 1:
            new = [i for i, e in enumerate(o.pool[0]) if e["level"] == p + 1]
            best = sorted(new, key=lambda i: -o.pool[0][i]["score"])[: cfg.topk]
            assert sorted(best) == sorted(o.frontier[0])
    pool = o.pool[0]
    assert len(pool) == cfg.topk + (cfg.D - 1) * cfg.topk ** 2 == 14          # all kept
    assert len(o.tree_tok[0]) == 15
    level = _check_tree_invariants(o, cfg)
    assert list(np.bincount(level)) == [1, 2, 4, 4, 4]
    # every candidate's score is the sum of the log-probabilities along its path
    for e in pool:
        total, a = 0.0, e
        while True:
            p = a["level"] - 1
            row = 0 if p == 0 else fronts[p].index(a["parent"])
            total += logps[p][row][a["tok"]]
            if a["parent"] == -1:
                break
            a = pool[a["parent"]]
        assert abs(total - e["score"]) < 1e-12
    # level-1 tokens are the two most likely tokens after the root, in rank order
    assert list(o.tree_tok[0][1:3]) == list(top_k(logps[0][0], 2))


def test_dynamic_selection_prunes_to_n_nodes_and_stays_ancestor_closed():
    cfg = ECFG.with_(D=3, topk=3, N=8)                      # pool 3 + 2 * 9 = 21 -> keep 7
    o = _eagle(cfg, HostWeights(WeightStore(cfg)))
    for p in range(cfg.D):
        o.draft(p)
        o.expand_tree(p)
    assert len(o.pool[0]) == 21 and len(o.tree_tok[0]) == 8
    _check_tree_invariants(o, cfg)
    vis = ancestor_matrix(o.tree_parent[0])
    assert vis[:, 0].all()


def test_medusa_heads_with_their_own_linear():
    """Section 3.1's Medusa head ends in a Linear per head.  Two pins that do not retype the
    oracle's product: (1) with every head's matrix equal to the target's LM head the result is the
    shared-head result; (2) with matrix i = the row pattern e_{(v + i) mod H} the logits are the
    head's own features read off in that order."""
    cfg = TINY_MEDUSA.with_(medusa_own_lm=True)
    base = HostWeights(WeightStore(TINY_MEDUSA))
    h = np.linspace(-1.0, 1.0, cfg.H)
    shared_logits, feats = KoalaOracle(TINY_MEDUSA, base).medusa_draft(h)

    class Same:
        def __call__(self, name):
            return base("lm_head") if name.endswith(".lm") else base(name)
    same_logits, same_feats = KoalaOracle(cfg, Same()).medusa_draft(h)
    assert np.array_equal(same_feats, feats)
    np.testing.assert_allclose(same_logits, shared_logits, rtol=0, atol=1e-12)   # summation order only

    class Pattern:
        def __call__(self, name):
            if name.endswith(".lm"):
                i = int(name.split(".")[1])
                w = np.zeros((cfg.V, cfg.H))
                w[np.arange(cfg.V), (np.arange(cfg.V) + i) % cfg.H] = 1.0
                return w
            return base(name)
    logits, f2 = KoalaOracle(cfg, Pattern()).medusa_draft(h)
    for i in range(cfg.n_medusa_heads):
        assert np.array_equal(logits[i], f2[i][(np.arange(cfg.V) + i) % cfg.H])
