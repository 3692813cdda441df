"""Whole-path parity on the tiny fp32 configurations: every call of every iteration is compared
with the oracle (free-running: both sides carry their own state from the same prompt)."""
import numpy as np
import pytest
import torch

from tests.harness import kv_to_oracle, make_pair, tok_list
from tests.parity import assert_close, check_argmax, check_topk
from workloads import TINY_EAGLE, TINY_MEDUSA
from workloads.generate import prompts

pytestmark = pytest.mark.gpu
EAGLE = 0


def _compare_state(eng, orc, cfg, what):
    S = eng.seq_len.cpu().numpy()
    assert list(S) == list(orc.seq_len), what
    bufs = eng.buffers()
    assert list(bufs["root_tok"].cpu().numpy()) == list(orc.root_tok), what
    for b in range(cfg.B):
        for l in range(cfg.L):
            assert_close(kv_to_oracle(eng.target_k, l, b, np.float64)[:S[b]], orc.target_k[l][b][:S[b]],
                         cfg.dtype, f"{what}: target K layer {l}")
            assert_close(kv_to_oracle(eng.target_v, l, b, np.float64)[:S[b]], orc.target_v[l][b][:S[b]],
                         cfg.dtype, f"{what}: target V layer {l}")
        n = int(bufs["n_pend"][b].item())
        assert n == orc.pend_hid[b].shape[0]
        assert_close(bufs["pend_hid"][b, :n].cpu().numpy(), orc.pend_hid[b], cfg.dtype, f"{what}: pending hidden")


def _run(cfg, flags, iters, chunk):
    eng, orc, _ = make_pair(cfg, flags)
    pr = prompts(cfg)
    chunk = min(chunk, cfg.N)
    eng.prefill(pr, chunk)
    orc.prefill(pr, chunk)
    assert eng.device_status() == 0
    _compare_state(eng, orc, cfg, "after prefill")
    passes = cfg.D if cfg.head_kind == EAGLE else 1
    k, N, B = cfg.topk, cfg.N, cfg.B
    emitted = [[] for _ in range(B)]
    def rows_of(b, p):
        if cfg.head_kind == EAGLE:
            return [b] if p == 0 else [b * k + i for i in range(k)]
        return [i * B + b for i in range(cfg.n_medusa_heads)]

    for it in range(iters):
        for p in range(passes):
            eng.koala_draft(p)
            orc.draft(p)
            bufs = eng.buffers()
            dl = bufs["draft_logits"].cpu().numpy()
            for b in range(B):
                assert_close(dl[rows_of(b, p)], orc.draft_logits[b], cfg.dtype,
                             f"iter {it} pass {p}: draft logits")
            eng.koala_expand_tree(p)
            orc.expand_tree(p)
            bufs = eng.buffers()
            tk = bufs["topk_tok"].cpu().numpy()
            for b in range(B):
                for j, r in enumerate(rows_of(b, p)):
                    check_topk(tk[r], orc.draft_logits[b][j], k, f"iter {it} pass {p} row {r}: top-k")
            if cfg.head_kind == EAGLE and p < passes - 1:
                assert bufs["frontier"].cpu().numpy().tolist() == [list(f) for f in orc.frontier]
        bufs = eng.buffers()
        for b in range(B):
            n = int(bufs["tree_n"][b].item())
            assert n == len(orc.tree_tok[b])
            assert bufs["tree_tok"][b, :n].cpu().numpy().tolist() == list(orc.tree_tok[b])
            assert bufs["tree_parent"][b, :n].cpu().numpy().tolist() == list(orc.tree_parent[b])
            if orc.tree_score[b] is not None:
                assert_close(bufs["tree_score"][b, :n].cpu().numpy(), orc.tree_score[b], cfg.dtype, "tree scores")
        eng.koala_verify(None)
        orc.verify()
        bufs = eng.buffers()
        for b in range(B):
            n = len(orc.tree_tok[b])
            assert_close(bufs["verify_logits"][b * N:b * N + n].cpu().numpy(), orc.verify_logits[b], cfg.dtype,
                         f"iter {it}: verify logits")
            assert_close(bufs["verify_hid"][b * N:b * N + n].cpu().numpy(), orc.verify_hid[b], cfg.dtype,
                         f"iter {it}: verify hidden")
            check_argmax(bufs["verify_tgt"][b * N:b * N + n].cpu().numpy(), orc.verify_logits[b], "verify arg-max")
        out = eng.koala_accept(None)
        ref_tok, ref_len = orc.accept()
        got_tok, got_len = tok_list(*out)
        assert got_len == ref_len and got_tok == ref_tok, f"iter {it}: accepted tokens"
        for b in range(B):
            emitted[b] += got_tok[b]
        _compare_state(eng, orc, cfg, f"after iteration {it}")
    assert eng.device_status() == 0
    # losslessness on the GPU side: the emitted stream is the oracle's greedy autoregressive stream
    ref = type(orc)(cfg, orc._w, dtype=orc.dt, static_tree=orc.static_tree)
    ref.prefill(pr, 64)
    ar = ref.ar_greedy(max(len(e) for e in emitted))
    for b in range(B):
        assert emitted[b] == ar[b][:len(emitted[b])]
    eng.close()


@pytest.mark.parametrize("flags", [0, 2], ids=["pdl", "no_pdl"])
def test_tiny_eagle_fp32_eight_iterations(flags):
    _run(TINY_EAGLE, flags, 8, 16)


def test_tiny_medusa_fp32():
    _run(TINY_MEDUSA.with_(S_max=192), 0, 6, 12)


def test_tiny_medusa_heads_with_their_own_linear():
    _run(TINY_MEDUSA.with_(S_max=192, medusa_own_lm=True, B=2, prompt_len=40, prompt_len_min=24, seed=6), 0, 5, 12)


def test_tiny_eagle_batch_of_three_ragged_prompts():
    cfg = TINY_EAGLE.with_(B=3, prompt_len=48, prompt_len_min=20, S_max=160, seed=4)
    _run(cfg, 0, 4, 15)
