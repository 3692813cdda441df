"""Per-call (teacher-forced) parity at the 7B / 13B shapes in bf16.

Both sides start from the same synthetic state (seeded random KV caches, hidden rows, tokens).
After every call the oracle's result is written over the GPU's, so that one excused near-tie
cannot cascade: each call is compared on identical inputs.
"""
import numpy as np
import pytest
import torch

from tests.harness import kv_to_oracle, make_pair, tok_list
from tests.parity import assert_close, check_argmax, check_topk
from workloads import T13_EAGLE, T33_EAGLE, T7_EAGLE, T7_MEDUSA, reduced
from workloads.generate import normal_tensor, prompt_lengths, random_kv, uniform_ints

pytestmark = pytest.mark.gpu
EAGLE = 0
DEV = "cuda:0"


def _seed_state(cfg, eng, orc, n_pend):
    """Same synthetic caches / pending rows on both sides."""
    B, N, H = cfg.B, cfg.N, cfg.H
    S = prompt_lengths(cfg).astype(np.int64)
    eng.target_k.copy_(random_kv(cfg, "target_k", cfg.L, DEV))
    eng.target_v.copy_(random_kv(cfg, "target_v", cfg.L, DEV))
    for l in range(cfg.L):
        for b in range(B):
            orc.target_k[l][b][...] = kv_to_oracle(eng.target_k, l, b, orc.dt)
            orc.target_v[l][b][...] = kv_to_oracle(eng.target_v, l, b, orc.dt)
    if cfg.head_kind == EAGLE:
        eng.draft_k.copy_(random_kv(cfg, "draft_k", cfg.K, DEV))
        eng.draft_v.copy_(random_kv(cfg, "draft_v", cfg.K, DEV))
        for j in range(cfg.K):
            for b in range(B):
                orc.draft_k[j][b][...] = kv_to_oracle(eng.draft_k, j, b, orc.dt)
                orc.draft_v[j][b][...] = kv_to_oracle(eng.draft_v, j, b, orc.dt)
    bufs = eng.buffers()
    eng.seq_len.copy_(torch.from_numpy(S.astype(np.int32)))
    hid = normal_tensor(3000 + cfg.seed, "pend_hid", (B, N, H), 1.0, 0.0, torch.float32, DEV)
    bufs["pend_hid"].copy_(hid)
    ptok = uniform_ints(3000 + cfg.seed, "pend_tok", B * N, 0, cfg.V).reshape(B, N)
    bufs["pend_tok"].copy_(torch.from_numpy(ptok))
    root = uniform_ints(3000 + cfg.seed, "root_tok", B, 0, cfg.V)
    bufs["root_tok"].copy_(torch.from_numpy(root))
    bufs["n_pend"].copy_(torch.from_numpy(np.asarray(n_pend, np.int32)))
    hid_h = hid.cpu().numpy()
    for b in range(B):
        orc.seq_len[b] = int(S[b])
        orc.root_tok[b] = int(root[b])
        orc.pend_hid[b] = hid_h[b, :n_pend[b]].astype(orc.dt)
        orc.pend_tok[b] = [int(t) for t in ptok[b, :n_pend[b] - 1]]
    return S


def _teacher_forced_iteration(cfg, flags=0):
    eng, orc, _ = make_pair(cfg, flags, oracle_dtype=np.float32, cache_host=False)
    B, N, k, V = cfg.B, cfg.N, cfg.topk, cfg.V
    n_pend = [1 + (b * 2 + 2) % min(cfg.D + 1, N) for b in range(B)]
    S = _seed_state(cfg, eng, orc, n_pend)
    passes = cfg.D if cfg.head_kind == EAGLE else 1
    excused = 0

    def rows_of(b, p):
        if cfg.head_kind == EAGLE:
            return [b] if p == 0 else [b * k + i for i in range(k)]
        return [i * B + b for i in range(cfg.n_medusa_heads)]

    for p in range(passes):
        eng.koala_draft(p)
        orc.draft(p)
        bufs = eng.buffers()
        dl = bufs["draft_logits"].cpu().numpy()
        for b in range(B):
            assert_close(dl[rows_of(b, p)], orc.draft_logits[b], cfg.dtype, f"pass {p}: draft logits")
        # features: compare, then continue from the oracle's
        feat = bufs["draft_feat"]
        for b in range(B):
            ref = orc.draft_feat[b]
            if cfg.head_kind == EAGLE:
                rows = [b * k] if p == 0 else [b * k + i for i in range(k)]
            else:
                rows = rows_of(b, p)
            assert_close(feat[rows].cpu().numpy(), ref, cfg.dtype, f"pass {p}: predicted features")
            feat[rows] = torch.from_numpy(np.ascontiguousarray(ref, dtype=np.float32)).to(DEV)
        eng.set_expand_mode(1)                       # top-k only
        eng.koala_expand_tree(p)
        bufs = eng.buffers()
        tk = bufs["topk_tok"].cpu().numpy()
        tl = bufs["topk_logp"].cpu().numpy()
        new_tok, new_lp = tk.copy(), tl.copy()
        for b in range(B):
            ref_logits = orc.draft_logits[b]
            m = ref_logits.max(axis=-1, keepdims=True)
            ref_lp = (ref_logits - m) - np.log(np.exp(ref_logits - m).sum(axis=-1, keepdims=True))
            for j, r in enumerate(rows_of(b, p)):
                excused += check_topk(tk[r], ref_logits[j], k, f"pass {p} row {r}: top-k")
                order = np.lexsort((np.arange(V), -ref_logits[j]))[:k]
                assert_close(tl[r], ref_lp[j][tk[r]], cfg.dtype, f"pass {p} row {r}: log-probabilities")
                new_tok[r], new_lp[r] = order, ref_lp[j][order]
        bufs["topk_tok"].copy_(torch.from_numpy(new_tok))
        bufs["topk_logp"].copy_(torch.from_numpy(new_lp.astype(np.float32)))
        eng.set_expand_mode(2)                       # tree bookkeeping from the oracle's top-k
        eng.koala_expand_tree(p)
        orc.expand_tree(p)
        bufs = eng.buffers()
        if cfg.head_kind == EAGLE and p < passes - 1:
            assert bufs["frontier"].cpu().numpy().tolist() == [list(f) for f in orc.frontier], f"pass {p}: frontier"
    eng.set_expand_mode(0)
    bufs = eng.buffers()
    for b in range(B):
        n = int(bufs["tree_n"][b].item())
        assert n == len(orc.tree_tok[b]) == N
        assert bufs["tree_tok"][b, :n].cpu().numpy().tolist() == list(orc.tree_tok[b])
        assert bufs["tree_parent"][b, :n].cpu().numpy().tolist() == list(orc.tree_parent[b])
        if orc.tree_score[b] is not None:
            assert np.array_equal(bufs["tree_score"][b, :n].cpu().numpy(), orc.tree_score[b].astype(np.float32))
    # ---- verify
    eng.koala_verify(None)
    orc.verify()
    bufs = eng.buffers()
    for b in range(B):
        assert_close(bufs["verify_hid"][b * N:(b + 1) * N].cpu().numpy(), orc.verify_hid[b], cfg.dtype,
                     "verify hidden states")
        assert_close(bufs["verify_logits"][b * N:(b + 1) * N].cpu().numpy(), orc.verify_logits[b], cfg.dtype,
                     "verify logits")
        excused += check_argmax(bufs["verify_tgt"][b * N:(b + 1) * N].cpu().numpy(), orc.verify_logits[b],
                                "verify arg-max")
    tgt = np.concatenate([orc.verify_tgt[b] for b in range(B)]).astype(np.int32)
    bufs["verify_tgt"].copy_(torch.from_numpy(tgt))
    # tree K/V written by verify (before compaction)
    for b in range(B):
        for l in (0, cfg.L - 1):
            sl = slice(int(S[b]), int(S[b]) + N)
            assert_close(kv_to_oracle(eng.target_k, l, b, np.float32)[sl], orc.target_k[l][b][sl], cfg.dtype,
                         f"tree keys layer {l}")
            assert_close(kv_to_oracle(eng.target_v, l, b, np.float32)[sl], orc.target_v[l][b][sl], cfg.dtype,
                         f"tree values layer {l}")
    # ---- accept with a forced schedule (random heads accept nothing by themselves)
    forced = np.asarray([1 + (3 * b + 2) % (cfg.D + 1) for b in range(B)], np.int32)
    out = eng.koala_accept(torch.from_numpy(forced).to(DEV))
    ref_tok, ref_len = orc.accept(list(forced))
    got_tok, got_len = tok_list(*out)
    assert got_len == ref_len and got_tok == ref_tok
    assert eng.seq_len.cpu().numpy().tolist() == orc.seq_len
    bufs = eng.buffers()
    assert bufs["root_tok"].cpu().numpy().tolist() == orc.root_tok
    for b in range(B):
        n = ref_len[b]
        assert int(bufs["n_pend"][b].item()) == n
        assert bufs["pend_tok"][b, :n - 1].cpu().numpy().tolist() == orc.pend_tok[b]
        assert_close(bufs["pend_hid"][b, :n].cpu().numpy(), orc.pend_hid[b], cfg.dtype, "accepted hidden rows")
        for l in (0, cfg.L - 1):
            sl = slice(int(S[b]), int(S[b]) + n)
            assert_close(kv_to_oracle(eng.target_k, l, b, np.float32)[sl], orc.target_k[l][b][sl], cfg.dtype,
                         f"compacted keys layer {l}")
            assert_close(kv_to_oracle(eng.target_v, l, b, np.float32)[sl], orc.target_v[l][b][sl], cfg.dtype,
                         f"compacted values layer {l}")
    assert eng.device_status() == 0
    eng.close()
    return excused


def test_t7_medusa_full_size():
    """The benchmark's configuration: 32 layers, 4 heads x K=2, static 64-node tree, context 512."""
    _teacher_forced_iteration(T7_MEDUSA)


def test_t7_medusa_heads_with_their_own_linear():
    """Each head streams a [V][H] matrix of its own for its B rows (two target layers keep it short)."""
    _teacher_forced_iteration(reduced(T7_MEDUSA, 2, medusa_own_lm=True))


@pytest.mark.parametrize("K", [1, 2, 4])
def test_t7_eagle_draft_and_verify(K):
    _teacher_forced_iteration(reduced(T7_EAGLE, 2, K=K))


def test_t7_eagle_full_depth():
    """The 7B configuration with the EAGLE-style head at full depth: 32 target layers, K = 2,
    dynamic tree of 60 nodes, context 1024."""
    _teacher_forced_iteration(T7_EAGLE)


def test_t13_eagle_full_depth_batch4_ragged():
    """The 13B configuration at full depth: 40 target layers, batch 4 with ragged contexts in
    [512, 2048], 64-node trees (256 rows per forward)."""
    _teacher_forced_iteration(T13_EAGLE)


@pytest.mark.parametrize("cfg", [reduced(T7_EAGLE, 3, K=2), reduced(T7_MEDUSA, 3), reduced(T13_EAGLE, 2, B=2)],
                         ids=["t7_eagle", "t7_medusa", "t13_eagle_batch2"])
def test_persistent_layer_kernel_path(cfg):
    """KOALA_F_LAYER_KERNEL: the same iteration with each layer's matrix multiplies and row-wise
    steps in one persistent launch (draft passes of 1..20 rows, verification of 60 / 64 / 128 rows)."""
    _teacher_forced_iteration(cfg, flags=4)


def test_t7_eagle_cuda_core_path_agrees():
    _teacher_forced_iteration(reduced(T7_EAGLE, 1, K=1, S_max=384, prompt_len=256), flags=1)


def test_t13_eagle_batch4_ragged():
    _teacher_forced_iteration(reduced(T13_EAGLE, 2))


@pytest.mark.parametrize("B,N", [(2, 64), (2, 60), (4, 64), (1, 128)], ids=["2x64", "2x60", "4x64", "1x128"])
def test_t7_shape_at_113_to_256_rows(B, N):
    """The 7B shape at 120 to 256 verification rows: the GEMMs run as CTA pairs over 512-row weight
    tiles; FFN 11008 = 21.5 tiles, so gate and up each end in a ragged tile and the second matrix
    starts in the middle of one."""
    _teacher_forced_iteration(reduced(T7_EAGLE, 2, K=1, B=B, N=N, S_max=640, prompt_len=384))


@pytest.mark.parametrize("K", [2, 6])
def test_t33_eagle_shape(K):
    """33B-shaped layers (hidden 6656, 52 heads, FFN 17920) with a deeper head; one target layer."""
    _teacher_forced_iteration(reduced(T33_EAGLE, 1, K=K, S_max=640, prompt_len=512))


def test_ragged_vocabulary_and_odd_top_k():
    """A vocabulary that is no multiple of the top-k kernel's parts or of the GEMM's 128-row tiles, k = 7."""
    _teacher_forced_iteration(reduced(T7_EAGLE, 1, K=1, V=5003 - 3, topk=7, N=40, S_max=384, prompt_len=256))
    _teacher_forced_iteration(reduced(T7_EAGLE, 1, K=1, V=32768, topk=16, D=2, N=64, S_max=384, prompt_len=256))
