"""CPU oracle for the draft-then-verify step of speculative decoding with K-layer draft heads.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow numpy restatement of what the paper's
method computes; it exists so that the CUDA library can be checked against it.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the product path
never does, and it shares no code with the CUDA sources.

What follows which passage of the paper (KOALA, arXiv 2408.08146):
  * autoregressive greedy decoding ............ Section 2.1, Eq. 1          (ar_greedy)
  * draft t tokens, verify them in one target
    forward giving q_1..q_{t+1} ............... Section 2.2, Eq. 2 and 3    (draft / verify)
  * greedy acceptance: keep a draft token only
    if it equals the target's greedy token .... Section 4.1 (setup)         (accept)
  * K-layer Medusa head (K x ResBlock -> Linear) Section 3.1                 (medusa_draft)
  * K-layer EAGLE head (Embedding -> Linear ->
    K x Decoder Layer -> LM Head) ............. Section 3.1                 (eagle_draft_pass)
  * acceptance length counts the tokens one
    target forward yields (bonus included) .... Section 4.1 (metrics)
The paper only names candidate trees and tree attention (Section 4.1 metrics, Section 5); the
definitions used here (node order, masks, scores, tie-breaks, static tree, forced lengths)
are the readings listed in the repository's design notes and are restated in each docstring.

Pins (tests/test_oracle_*.py): decoder stack against the `transformers` Llama implementation;
tree verification against per-path causal forwards; chain tree against plain prefill;
speculative output stream against ar_greedy (losslessness); planted paths; cache after
acceptance against a direct prefill; Medusa K=0 / zero-weight / composition cases; EAGLE fc
selector cases and tree-vs-chain drafting; top-k and tree selection against brute-force sorts.
PARITY UNPINNED: the overall wiring of the EAGLE-style head (which token is paired with which
hidden state, and that a tree node's input feature is its parent's predicted feature) has no
external truth in the paper; only its parts are pinned.

Precision: every array is `dtype` (float64 by default; float32 for the 7B/13B shapes, whose
weights are the bf16-rounded values upcast exactly).
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np

EAGLE = 0
MEDUSA = 1


# ----------------------------------------------------------------------------------------------
# Elementary operations (closed forms)
# ----------------------------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """g * x / sqrt(mean(x^2) + eps) over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return g * (x / np.sqrt(ms + eps))


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary position embedding, half-split pairing (i, i + dh/2).

    x: [n, n_heads, dh]; pos: [n] absolute 0-based token positions;
    theta_i = base ** (-2 i / dh), i = 0 .. dh/2 - 1.
    """
    dh = x.shape[-1]
    half = dh // 2
    inv = base ** (-(np.arange(half, dtype=np.float64) * 2.0) / dh)
    ang = pos.astype(np.float64)[:, None] * inv[None, :]           # [n, half]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def masked_softmax(scores: np.ndarray, visible: np.ndarray) -> np.ndarray:
    """Row-wise softmax over the visible entries; hidden entries contribute exactly 0."""
    s = np.where(visible, scores, -np.inf)
    m = np.max(s, axis=-1, keepdims=True)
    e = np.where(visible, np.exp(s - m), 0.0)
    return e / np.sum(e, axis=-1, keepdims=True)


def log_softmax(z: np.ndarray) -> np.ndarray:
    m = np.max(z, axis=-1, keepdims=True)
    return (z - m) - np.log(np.sum(np.exp(z - m), axis=-1, keepdims=True))


def top_k(values: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries: larger value first, then the smaller index."""
    order = np.lexsort((np.arange(values.shape[0]), -values))
    return order[:k].astype(np.int64)


def sample_index(w: np.ndarray, u: float) -> int:
    """Inverse-CDF draw in index order from non-negative weights: the smallest j with
    w_0 + .. + w_j > u * sum(w), u in [0, 1) (rounding can leave none: then the last j with w_j > 0)."""
    c = np.cumsum(np.asarray(w, dtype=np.float64))
    j = int(np.searchsorted(c, u * c[-1], side="right"))
    if j >= len(c):
        j = int(np.nonzero(np.asarray(w) > 0)[0][-1])
    return j


def speculative_sampling_step(d, q, drafted, u_accept, u_bonus):
    """Acceptance of a chain of t drafted tokens by speculative sampling (Section 2.2, the
    paragraph after Eq. 3).  d[i], q[i]: draft and target distributions at chain position i
    (q has t + 1 rows); drafted[i] was drawn from d[i].  Token i is accepted with probability
    min(1, q_i(x_i) / d_i(x_i)), i.e. iff u_accept[i] * d_i(x_i) < q_i(x_i); the first rejected
    position f is redrawn from norm(max(0, q_f - d_f)) and the rest discarded; if all t are accepted
    one more token is drawn from q_{t+1}.  Both draws use u_bonus.  Returns (accepted count, the
    extra token)."""
    t = len(drafted)
    for i in range(t):
        x = int(drafted[i])
        if not (u_accept[i] * d[i][x] < q[i][x]):
            return i, sample_index(np.maximum(0.0, np.asarray(q[i], np.float64) - np.asarray(d[i], np.float64)), u_bonus)
    return t, sample_index(q[t], u_bonus)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of float32 values to bfloat16 (8 significant bits), returned as float32.

    Storage rounding of a bf16 KV cache: the paper does not state a numeric precision (Section 4.1
    gives none); the bf16 configurations store weights and caches in bf16, and a value is rounded
    to the storage type when it is written.
    """
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def argmax_first(values: np.ndarray) -> int:
    """Index of the maximum; the smallest index among equal maxima."""
    return int(np.argmax(values))


# ----------------------------------------------------------------------------------------------
# Tree helpers
# ----------------------------------------------------------------------------------------------

def tree_levels(parent: Sequence[int]) -> np.ndarray:
    level = np.zeros(len(parent), dtype=np.int64)
    for u in range(1, len(parent)):
        assert 0 <= parent[u] < u, "parents must precede children"
        level[u] = level[parent[u]] + 1
    return level


def ancestor_matrix(parent: Sequence[int]) -> np.ndarray:
    """vis[u, v] = True iff v is u itself or an ancestor of u."""
    n = len(parent)
    vis = np.zeros((n, n), dtype=bool)
    for u in range(n):
        v = u
        while v >= 0:
            vis[u, v] = True
            v = parent[v]
    return vis


# ----------------------------------------------------------------------------------------------
# The oracle proper
# ----------------------------------------------------------------------------------------------

class KoalaOracle:
    """State and the five steps (draft, expand_tree, verify, accept; init is the constructor).

    cfg: an object with fields L, H, n_heads, head_dim, F, V, K, D, topk, N, B, S_max,
         head_kind, n_medusa_heads, rms_eps, rope_base.
    weight: callable name -> numpy array ([out][in] matrices; names as in the workload module).
    static_tree: (parent, level, rank) arrays for the Medusa-style static topology.
    kv_round: optional storage rounding applied to keys and values as they enter a cache.
    """

    def __init__(self, cfg, weight: Callable[[str], np.ndarray], dtype=np.float64,
                 static_tree=None, kv_round: Optional[Callable[[np.ndarray], np.ndarray]] = None):
        self.cfg = cfg
        self.dt = dtype
        self.kv_round = kv_round        # storage rounding of the caches (round_to_bf16 for bf16 caches)
        self._w = weight
        B, L, K = cfg.B, cfg.L, cfg.K
        shape = (cfg.S_max, cfg.n_heads, cfg.head_dim)
        self.target_k = [[np.zeros(shape, dtype) for _ in range(B)] for _ in range(L)]
        self.target_v = [[np.zeros(shape, dtype) for _ in range(B)] for _ in range(L)]
        n_draft_kv = K if cfg.head_kind == EAGLE else 0
        self.draft_k = [[np.zeros(shape, dtype) for _ in range(B)] for _ in range(n_draft_kv)]
        self.draft_v = [[np.zeros(shape, dtype) for _ in range(B)] for _ in range(n_draft_kv)]
        self.chain_d = [dict() for _ in range(cfg.B)]   # [b][level] draft distribution of a sampled chain
        self.alpha_hits = [0] * cfg.N      # [n-1]: iterations whose n-th draft token was accepted
        self.alpha_trials = [0] * cfg.N    # [n-1]: iterations that offered an n-th draft token after n-1 accepted
        self.seq_len = [0] * B                  # tokens held by the target cache
        self.root_tok = [0] * B                 # x_S: the token the next tree is rooted at
        self.pend_hid: List[np.ndarray] = [np.zeros((0, cfg.H), dtype) for _ in range(B)]
        self.pend_tok: List[List[int]] = [[] for _ in range(B)]
        self.static_tree = static_tree
        # per-iteration results
        self.draft_logits: List[Optional[np.ndarray]] = [None] * B
        self.draft_feat: List[Optional[np.ndarray]] = [None] * B
        self.pool: List[list] = [[] for _ in range(B)]       # candidates: level, parent, rank, tok, score
        self.frontier: List[list] = [[] for _ in range(B)]   # candidate ids expanded by the next pass
        self.feat_of: List[dict] = [{} for _ in range(B)]
        self.row_of: List[dict] = [{} for _ in range(B)]
        self.tree_tok: List[Optional[np.ndarray]] = [None] * B
        self.tree_parent: List[Optional[np.ndarray]] = [None] * B
        self.tree_score: List[Optional[np.ndarray]] = [None] * B
        self.verify_logits: List[Optional[np.ndarray]] = [None] * B
        self.verify_hid: List[Optional[np.ndarray]] = [None] * B
        self.verify_tgt: List[Optional[np.ndarray]] = [None] * B

    def W(self, name: str) -> np.ndarray:
        return np.asarray(self._w(name), dtype=self.dt)

    # ------------------------------------------------------------------ decoder layer
    def decoder_layer(self, x: np.ndarray, pos: np.ndarray, slots: np.ndarray,
                      visible: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                      prefix: str) -> np.ndarray:
        """One pre-norm Llama-style layer over n new rows of one sequence.

        x [n, H]; row i has RoPE position pos[i]; its key/value are stored at cache slot slots[i]
        first, then row i attends to the cache slots j < T with visible[i, j] (T = visible.shape[1]).
        x <- x + Wo Attn(RMSNorm(x));  x <- x + Wdown (SiLU(Wgate n) * Wup n), n = RMSNorm(x);
        Attn = softmax(q k^T / sqrt(dh)) v per head, q and k rotated by RoPE.
        """
        c = self.cfg
        n, T = x.shape[0], visible.shape[1]
        h = rmsnorm(x, self.W(prefix + "attn_norm"), c.rms_eps)
        q = (h @ self.W(prefix + "wq").T).reshape(n, c.n_heads, c.head_dim)
        k = (h @ self.W(prefix + "wk").T).reshape(n, c.n_heads, c.head_dim)
        v = (h @ self.W(prefix + "wv").T).reshape(n, c.n_heads, c.head_dim)
        q = rope(q, pos, c.rope_base)
        k = rope(k, pos, c.rope_base)
        if self.kv_round is not None:           # the caches hold values in their storage type
            k = self.kv_round(k).astype(self.dt)
            v = self.kv_round(v).astype(self.dt)
        k_cache[slots] = k
        v_cache[slots] = v
        scale = 1.0 / np.sqrt(float(c.head_dim))
        attn = np.empty((n, c.n_heads, c.head_dim), dtype=self.dt)
        for hd in range(c.n_heads):
            s = (q[:, hd, :] @ k_cache[:T, hd, :].T) * scale
            attn[:, hd, :] = masked_softmax(s, visible) @ v_cache[:T, hd, :]
        x = x + attn.reshape(n, c.H) @ self.W(prefix + "wo").T
        h = rmsnorm(x, self.W(prefix + "ffn_norm"), c.rms_eps)
        act = silu(h @ self.W(prefix + "w_gate").T) * (h @ self.W(prefix + "w_up").T)
        return x + act @ self.W(prefix + "w_down").T

    # ------------------------------------------------------------------ target forward (Eq. 3)
    def target_forward(self, b: int, tok: np.ndarray, parent: np.ndarray):
        """Target forward over the nodes of one sequence's tree, on top of its cached context.

        Node u sits at position S + level(u), its key/value at slot S + u, and it attends to the
        S context tokens, its ancestors and itself.  Returns (logits [n, V], hid [n, H]) where
        hid is the output of the final RMSNorm, i.e. the LM head's input.
        """
        c = self.cfg
        S = self.seq_len[b]
        n = len(tok)
        assert S + n <= c.S_max, "KV capacity exceeded"
        level = tree_levels(parent)
        visible = np.concatenate([np.ones((n, S), dtype=bool), ancestor_matrix(parent)], axis=1)
        x = self.W("embed")[np.asarray(tok, dtype=np.int64)]
        pos = S + level
        slots = S + np.arange(n)
        for l in range(c.L):
            x = self.decoder_layer(x, pos, slots, visible, self.target_k[l][b],
                                   self.target_v[l][b], f"layers.{l}.")
        hid = rmsnorm(x, self.W("final_norm"), c.rms_eps)
        logits = hid @ self.W("lm_head").T
        return logits, hid

    # ------------------------------------------------------------------ Medusa-style draft
    def medusa_draft(self, h_last: np.ndarray):
        """Head i (0-based): x <- h_last; K times x <- x + SiLU(W_ij x + b_ij); logits = LM(x).

        Non-autoregressive: all heads read the same hidden state.  LM is the target's LM head,
        shared by the heads, or - cfg.medusa_own_lm, Section 3.1's head as drawn: K x ResBlock
        followed by a Linear of its own - the head's own [V, H] matrix "medusa.i.lm".
        Returns (logits [n_medusa_heads, V], features); head i ranks the token at tree level i+1.
        """
        c = self.cfg
        feats = []
        for i in range(c.n_medusa_heads):
            x = h_last.astype(self.dt)
            for j in range(c.K):
                x = x + silu(self.W(f"medusa.{i}.{j}.w") @ x + self.W(f"medusa.{i}.{j}.b"))
            feats.append(x)
        feats = np.stack(feats, axis=0)
        if getattr(c, "medusa_own_lm", False):
            logits = np.stack([self.W(f"medusa.{i}.lm") @ feats[i] for i in range(c.n_medusa_heads)], axis=0)
            return logits, feats
        return feats @ self.W("lm_head").T, feats

    # ------------------------------------------------------------------ EAGLE-style draft pass
    def eagle_forward(self, b: int, feat_in: np.ndarray, tok: np.ndarray, pos: np.ndarray,
                      slots: np.ndarray, visible: np.ndarray):
        """z = W_fc [feature ; E[token]] + b_fc, then K decoder layers with the head's own KV cache.

        Returns (f_hat [n, H], logits [n, V]): f_hat is the predicted next feature (no norm after
        the last layer) and logits = LM_head(f_hat), with the target's own embedding and LM head.
        """
        c = self.cfg
        emb = self.W("embed")[np.asarray(tok, dtype=np.int64)]
        z = np.concatenate([feat_in, emb], axis=1) @ self.W("fc_w").T + self.W("fc_b")
        for j in range(c.K):
            z = self.decoder_layer(z, pos, slots, visible, self.draft_k[j][b], self.draft_v[j][b],
                                   f"draft.{j}.")
        return z, z @ self.W("lm_head").T

    # ------------------------------------------------------------------ draft (Eq. 2)
    def draft(self, p: int):
        """Draft pass p.  Medusa-style heads have the single pass 0.

        EAGLE-style, pass 0: the rows are the positions accepted by the last iteration
        (S - l_prev .. S - 1), each pairing the target's hidden state at position j with the
        token at position j + 1 (the last row pairs h_{S-1} with the root x_S); their keys and
        values extend the head's cache to length S and the last row's logits rank x_{S+1}.
        Pass p >= 1: the rows are the k frontier candidates of level p, each pairing its parent's
        predicted feature with its own token at head position S + p - 1; row i of the pass uses
        cache slot S + (p-1) k + i and attends to the S context entries, to the rows of its
        frontier ancestors and to itself.
        """
        c = self.cfg
        for b in range(c.B):
            S = self.seq_len[b]
            if c.head_kind == MEDUSA:
                assert p == 0
                self.draft_logits[b], self.draft_feat[b] = self.medusa_draft(self.pend_hid[b][-1])
                continue
            if p == 0:
                hid = self.pend_hid[b]
                n = hid.shape[0]
                toks = np.asarray(list(self.pend_tok[b]) + [self.root_tok[b]], dtype=np.int64)
                assert len(toks) == n and n >= 1
                pos = np.arange(S - n, S)
                visible = np.concatenate([np.ones((n, S - n), dtype=bool),
                                          np.tril(np.ones((n, n), dtype=bool))], axis=1)
                f_hat, logits = self.eagle_forward(b, hid, toks, pos, pos, visible)
                self.draft_feat[b], self.draft_logits[b] = f_hat[-1:], logits[-1:]
                self.pool[b] = []
                self.frontier[b] = []
                self.feat_of[b] = {-1: f_hat[-1]}     # candidate id -> feature it predicted
                self.row_of[b] = {}                   # candidate id -> row among the tree slots
            else:
                pool, fr = self.pool[b], self.frontier[b]
                k = len(fr)
                base = (p - 1) * k
                feat_in = np.stack([self.feat_of[b][pool[cid]["parent"]] for cid in fr], axis=0)
                toks = np.asarray([pool[cid]["tok"] for cid in fr], dtype=np.int64)
                pos = np.full(k, S + p - 1)
                slots = S + base + np.arange(k)
                vis_tree = np.zeros((k, base + k), dtype=bool)
                for i, cid in enumerate(fr):
                    self.row_of[b][cid] = base + i
                    a = cid
                    while a != -1:
                        vis_tree[i, self.row_of[b][a]] = True
                        a = pool[a]["parent"]
                visible = np.concatenate([np.ones((k, S), dtype=bool), vis_tree], axis=1)
                f_hat, logits = self.eagle_forward(b, feat_in, toks, pos, slots, visible)
                for i, cid in enumerate(fr):
                    self.feat_of[b][cid] = f_hat[i]
                self.draft_feat[b], self.draft_logits[b] = f_hat, logits

    # ------------------------------------------------------------------ tree expansion
    def expand_tree(self, p: int, u_draft=None):
        """Top-k expansion after draft pass p.

        u_draft (one uniform per sequence, chain drafts only: k = 1): the level's token is drawn
        from softmax(logits) by `sample_index` instead of being the arg-max (Section 2.2: the
        draft distributions d_i govern the sampling of the drafted tokens); the distribution is
        kept in chain_d[b][p] for `accept_sampled`.

        Dynamic tree (EAGLE-style): each row's k best tokens are taken from its logits (larger
        logit first, then smaller id); a candidate's score is its parent's score plus the token's
        natural-log softmax probability (root: 0).  Pass 0 yields k level-1 candidates, which all
        become the level-1 frontier (slot = rank).  Pass p >= 1 yields k*k level-(p+1) candidates
        in (frontier slot, rank) order; for p < D-1 the k best of them (score descending, then
        pool order) form the next frontier in that order.  After pass D-1 the N-1 best candidates
        of the whole pool (same order rule) plus the root form the tree; nodes are numbered by
        (level, parent's node number, rank).
        Static tree (Medusa-style): the node with (level d, rank r) takes the r-th best token of
        head d-1; the topology is fixed.
        """
        c = self.cfg
        for b in range(c.B):
            if c.head_kind == MEDUSA:
                parent, level, rank = self.static_tree
                tok = np.zeros(len(parent), dtype=np.int64)
                tok[0] = self.root_tok[b]
                best = [top_k(self.draft_logits[b][i], c.topk) for i in range(c.n_medusa_heads)]
                for u in range(1, len(parent)):
                    tok[u] = best[level[u] - 1][rank[u]]
                self.tree_tok[b] = tok
                self.tree_parent[b] = np.asarray(parent, dtype=np.int64)
                self.tree_score[b] = None
                continue
            logits = self.draft_logits[b]
            logp = log_softmax(logits)
            pool = self.pool[b]
            first_new = len(pool)
            parents = [-1] if p == 0 else list(self.frontier[b])
            for i, par in enumerate(parents):
                base_score = self.dt(0.0) if par == -1 else pool[par]["score"]
                picks = top_k(logits[i], c.topk)
                if u_draft is not None:
                    assert c.topk == 1, "drafted tokens are sampled on chains only"
                    dist = np.exp(logp[i])
                    self.chain_d[b][p] = dist
                    picks = [sample_index(dist, float(u_draft[b]))]
                for r, t in enumerate(picks):
                    pool.append({"level": p + 1, "parent": par, "rank": r, "tok": int(t),
                                 "score": self.dt(base_score + logp[i][t])})
            new_ids = list(range(first_new, len(pool)))
            if p < c.D - 1:
                if p == 0:
                    self.frontier[b] = new_ids
                else:
                    self.frontier[b] = sorted(new_ids, key=lambda i: (-pool[i]["score"], i))[: c.topk]
            else:
                self._finalise_tree(b)

    def _finalise_tree(self, b: int):
        c = self.cfg
        pool = self.pool[b]
        keep = sorted(range(len(pool)), key=lambda i: (-pool[i]["score"], i))[: c.N - 1]
        node_of = {-1: 0}
        tok, parent, score = [self.root_tok[b]], [-1], [self.dt(0.0)]
        max_level = max((pool[i]["level"] for i in keep), default=0)
        for lvl in range(1, max_level + 1):
            here = [i for i in keep if pool[i]["level"] == lvl]
            assert all(pool[i]["parent"] in node_of for i in here), "kept set must be ancestor-closed"
            here.sort(key=lambda i: (node_of[pool[i]["parent"]], pool[i]["rank"]))
            for i in here:
                node_of[i] = len(tok)
                tok.append(pool[i]["tok"])
                parent.append(node_of[pool[i]["parent"]])
                score.append(pool[i]["score"])
        assert len(tok) == 1 + len(keep)
        self.tree_tok[b] = np.asarray(tok, dtype=np.int64)
        self.tree_parent[b] = np.asarray(parent, dtype=np.int64)
        self.tree_score[b] = np.asarray(score, dtype=self.dt)

    # ------------------------------------------------------------------ verify (Eq. 3)
    def verify(self, caller_tree=None):
        """One target forward over every sequence's tree; tgt[u] = greedy token after node u.

        caller_tree: optional list (one per sequence) of (tok, parent) replacing the drafted tree
        (a chain for prompt ingestion, a single node for plain autoregressive decoding).
        """
        for b in range(self.cfg.B):
            if caller_tree is not None:
                tok, parent = caller_tree[b]
                self.tree_tok[b] = np.asarray(tok, dtype=np.int64)
                self.tree_parent[b] = np.asarray(parent, dtype=np.int64)
            logits, hid = self.target_forward(b, self.tree_tok[b], self.tree_parent[b])
            self.verify_logits[b], self.verify_hid[b] = logits, hid
            self.verify_tgt[b] = np.asarray([argmax_first(r) for r in logits], dtype=np.int64)

    # ------------------------------------------------------------------ accept + compaction
    def _commit_path(self, b: int, path, bonus: int, last_has_child: bool):
        """Bookkeeping shared by the acceptance rules: counters, cache compaction, pending rows."""
        c = self.cfg
        tok = self.tree_tok[b]
        ell = len(path)
        # position-wise acceptance (the n-alpha metric of Section 4.1, metrics): the n-th draft
        # token on the walked path was tried if the walk reached depth n-1 and that node has a
        # child; it was hit if the walk went on to depth n
        while len(self.alpha_hits) < ell:           # a caller's tree may be deeper than N
            self.alpha_hits.append(0)
            self.alpha_trials.append(0)
        for n in range(1, ell):
            self.alpha_hits[n - 1] += 1
            self.alpha_trials[n - 1] += 1
        if last_has_child:
            self.alpha_trials[ell - 1] += 1
        S = self.seq_len[b]
        for l in range(c.L):
            for cache in (self.target_k[l][b], self.target_v[l][b]):
                fresh = np.zeros_like(cache)
                fresh[:S] = cache[:S]
                fresh[S:S + ell] = cache[S + np.asarray(path)]
                cache[...] = fresh
        self.pend_hid[b] = self.verify_hid[b][np.asarray(path)].copy()
        self.pend_tok[b] = [int(tok[v]) for v in path[1:]]
        self.seq_len[b] = S + ell
        self.root_tok[b] = bonus
        return [int(tok[v]) for v in path[1:]] + [bonus], ell

    def reset_alpha(self):
        """Clears the position-wise acceptance counters (they also count forced prompt chunks)."""
        self.alpha_hits = [0] * self.cfg.N
        self.alpha_trials = [0] * self.cfg.N

    def accept(self, forced_len: Optional[Sequence[int]] = None):
        """Greedy acceptance of the longest matching root path, then cache compaction.

        Walk from the root: move to the (lowest-numbered) child whose token equals the target's
        greedy token at the current node; stop when there is none.  The path has l nodes; the
        iteration emits the path's tokens after the root followed by the bonus token
        tgt[last node] (l tokens), and the bonus becomes the next root.
        forced_len[b] = f > 0 replaces the stopping rule: where no child matches, step to the
        lowest-numbered child, until the path has f nodes or a leaf is reached.
        The accepted nodes' keys/values move to slots S .. S+l-1 of every target layer (built
        here as a fresh array), and seq_len grows by l.  The accepted hidden rows and tokens
        are kept as the next draft pass 0's input.
        Returns (emitted tokens per sequence, accepted length per sequence).
        """
        c = self.cfg
        out_tok, out_len = [], []
        for b in range(c.B):
            tok, parent, tgt = self.tree_tok[b], self.tree_parent[b], self.verify_tgt[b]
            n = len(tok)
            children = [[] for _ in range(n)]
            for u in range(1, n):
                children[parent[u]].append(u)
            f = int(forced_len[b]) if forced_len is not None else 0
            path = [0]
            u = 0
            while True:
                if f > 0 and len(path) >= f:
                    break
                nxt = next((ch for ch in children[u] if tok[ch] == tgt[u]), None)
                if nxt is None and f > 0 and children[u]:
                    nxt = children[u][0]
                if nxt is None:
                    break
                path.append(nxt)
                u = nxt
            toks_b, ell = self._commit_path(b, path, int(tgt[u]), bool(children[u]))
            out_tok.append(toks_b)
            out_len.append(ell)
        return out_tok, out_len

    def accept_sampled(self, u_accept, u_bonus):
        """Speculative-sampling acceptance of a chain tree (Section 2.2; temperature 1): position i
        of the chain is judged with q_i = softmax of the target's logits at node i-1 and the draft
        distribution kept by `expand_tree(p, u_draft)`; see `speculative_sampling_step`.
        u_accept[b][i], u_bonus[b]: uniforms in [0, 1).  Returns (tokens, lengths) like `accept`."""
        c = self.cfg
        out_tok, out_len = [], []
        for b in range(c.B):
            tok, parent = self.tree_tok[b], self.tree_parent[b]
            n = len(tok)
            assert all(int(parent[i]) == i - 1 for i in range(n)), "speculative sampling is defined on chains"
            q = np.exp(log_softmax(self.verify_logits[b][:n]))
            d = [self.chain_d[b][i] for i in range(n - 1)]
            a, bonus = speculative_sampling_step(d, q, [int(t) for t in tok[1:]], u_accept[b], float(u_bonus[b]))
            toks_b, ell = self._commit_path(b, list(range(a + 1)), int(bonus), a + 1 < n)
            out_tok.append(toks_b)
            out_len.append(ell)
        return out_tok, out_len

    # ------------------------------------------------------------------ drivers used by tests
    def prefill(self, prompts: Sequence[Sequence[int]], chunk: int):
        """Ingest the prompts as chain trees with full forced acceptance.

        Every sequence's prompt is cut into the same number of chunks (at most `chunk` tokens
        each).  For an EAGLE-style head the head's cache is filled the same way: after each chunk
        but the last, the next prompt token is set as the root and draft pass 0 runs over the
        chunk; the last chunk's root is the target's own greedy token, and its pass 0 is the
        first iteration's.
        """
        c = self.cfg
        n_chunks = max(-(-len(p) // chunk) for p in prompts)
        parts = [np.array_split(np.asarray(p, dtype=np.int64), n_chunks) for p in prompts]
        for ci in range(n_chunks):
            trees = [(parts[b][ci], np.arange(-1, len(parts[b][ci]) - 1)) for b in range(c.B)]
            self.verify(trees)
            self.accept([len(t[0]) for t in trees])
            if c.head_kind == EAGLE and ci + 1 < n_chunks:
                for b in range(c.B):
                    self.root_tok[b] = int(parts[b][ci + 1][0])
                self.draft(0)

    def step(self, forced_len=None):
        """One whole iteration: D x (draft, expand), verify, accept."""
        c = self.cfg
        passes = c.D if c.head_kind == EAGLE else 1
        for p in range(passes):
            self.draft(p)
            self.expand_tree(p)
        self.verify()
        return self.accept(forced_len)

    def ar_greedy(self, n_tokens: int):
        """Plain greedy autoregressive decoding (Eq. 1): one single-node verify per token."""
        c = self.cfg
        out = [[] for _ in range(c.B)]
        for _ in range(n_tokens):
            self.verify([(np.asarray([self.root_tok[b]]), np.asarray([-1])) for b in range(c.B)])
            toks, _ = self.accept()
            for b in range(c.B):
                out[b].extend(toks[b])
        return out
