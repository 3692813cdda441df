"""Speculative sampling on chain drafts (Section 2.2): the CUDA path against the oracle with the
same uniforms.  Every stochastic decision compares a uniform with a floating-point quantity, so
both sides must decide on the same numbers: after each forward the logits are compared within the
usual tolerance and the oracle's (as fp32) are written over the GPU's.  What is left is fp32 against
fp64 arithmetic on identical inputs; the tests check, on the oracle's side, that no decision of the
run lies within 2e-6 (draws, of the total mass) / 1e-5 (acceptance, relative) of its boundary, and
then demand identical tokens and lengths."""
import numpy as np
import pytest
import torch

from oracle.koala_oracle import log_softmax
from tests.harness import make_pair, tok_list
from tests.parity import assert_close
from workloads import T7_EAGLE, TINY_EAGLE, reduced
from workloads.generate import prompts

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _margin_ok(w, u, j):
    """u * sum(w) is not within 2e-6 * sum(w) of the CDF boundaries around index j."""
    c = np.cumsum(np.asarray(w, np.float64))
    t = u * c[-1]
    lo = c[j - 1] if j > 0 else 0.0
    return (t - lo) > 2e-6 * c[-1] and (c[j] - t) > 2e-6 * c[-1]


def _uniforms(seed, B, D):
    rng = np.random.default_rng(seed)
    return rng.random((B, D)).astype(np.float32), rng.random((B, D)).astype(np.float32), rng.random(B).astype(np.float32)


def _iteration(cfg, eng, orc, seed, check_dist):
    B, D = cfg.B, cfg.D
    u_d, u_a, u_b = _uniforms(seed, B, D)
    t_ud = torch.from_numpy(u_d).to(DEV)
    eng.koala_set_sampling(t_ud)
    for p in range(D):
        eng.koala_draft(p)
        orc.draft(p)
        dl = eng.buffers()["draft_logits"]
        for b in range(B):
            assert_close(dl[b:b + 1].cpu().numpy(), orc.draft_logits[b][:1], cfg.dtype, f"pass {p}: draft logits")
            orc.draft_logits[b] = orc.draft_logits[b].astype(np.float32).astype(orc.dt)
            dl[b] = torch.from_numpy(orc.draft_logits[b][0].astype(np.float32)).to(DEV)
            # the next pass continues from the oracle's predicted feature as well
            eng.buffers()["draft_feat"][b] = torch.from_numpy(orc.draft_feat[b][-1].astype(np.float32)).to(DEV)
        eng.koala_expand_tree(p)
        orc.expand_tree(p, u_draft=u_d[:, p])
        for b in range(B):
            d = orc.chain_d[b][p]
            assert _margin_ok(d, float(u_d[b, p]), int(orc.pool[b][-1]["tok"])), "seed lands on a boundary: pick another"
    bufs = eng.buffers()
    for b in range(B):
        n = len(orc.tree_tok[b])
        assert bufs["tree_tok"][b, :n].cpu().tolist() == [int(x) for x in orc.tree_tok[b]]
        assert bufs["tree_parent"][b, :n].cpu().tolist() == list(range(-1, n - 1))
    eng.koala_verify(None)
    orc.verify()
    vl = eng.buffers()["verify_logits"]
    for b in range(B):
        n = len(orc.tree_tok[b])
        assert_close(vl[b * cfg.N:b * cfg.N + n].cpu().numpy(), orc.verify_logits[b][:n], cfg.dtype, "verify logits")
        orc.verify_logits[b] = orc.verify_logits[b].astype(np.float32).astype(orc.dt)
        vl[b * cfg.N:b * cfg.N + n] = torch.from_numpy(orc.verify_logits[b][:n].astype(np.float32)).to(DEV)
    for b in range(B):                      # margins of the accept / redraw decisions, oracle side
        n = len(orc.tree_tok[b])
        q = np.exp(log_softmax(orc.verify_logits[b][:n].astype(np.float64)))
        for i in range(1, n):
            x = int(orc.tree_tok[b][i]); d = orc.chain_d[b][i - 1]
            lhs, rhs = float(u_a[b, i - 1]) * d[x], q[i - 1][x]
            assert abs(lhs - rhs) > 1e-5 * max(lhs, rhs), "seed lands on a boundary: pick another"
    got = tok_list(*eng.koala_accept_sampled(torch.from_numpy(u_a).to(DEV), torch.from_numpy(u_b).to(DEV)))
    ref = orc.accept_sampled(u_a, u_b)
    assert list(got[1]) == list(ref[1]), (got, ref)
    assert [list(x) for x in got[0]] == [list(x) for x in ref[0]], (got, ref)
    assert eng.seq_len.cpu().tolist() == orc.seq_len
    return got[1]


def test_tiny_chain_sampling_free_running():
    cfg = TINY_EAGLE.with_(topk=1, D=4, N=5, S_max=192, B=2, prompt_len=40, prompt_len_min=30, seed=9)
    eng, orc, _ = make_pair(cfg)
    pr = prompts(cfg)
    eng.prefill(pr, cfg.N)
    orc.prefill(pr, cfg.N)
    eng.koala_accept_stats(1, reset=True)
    orc.reset_alpha()
    lens = []
    for it in range(8):
        lens += _iteration(cfg, eng, orc, 100 + it, True)
    assert eng.koala_accept_stats(cfg.N) == (orc.alpha_hits[:cfg.N], orc.alpha_trials[:cfg.N])
    assert eng.device_status() == 0
    # back to greedy drafts and greedy acceptance on the same context
    eng.koala_set_sampling(None)
    got = tok_list(*eng.step())
    ref = orc.step()
    assert list(got[0]) == ref[0] and list(got[1]) == ref[1]
    eng.close()


def test_t7_shape_chain_sampling_one_iteration():
    """Vocabulary 32000, bf16: the kept draft distribution and one sampled iteration."""
    cfg = reduced(T7_EAGLE, 2, K=1, topk=1, D=3, N=4, S_max=384, prompt_len=256)
    eng, orc, _ = make_pair(cfg, oracle_dtype=np.float32, cache_host=False)
    pr = prompts(cfg)
    eng.prefill(pr, cfg.N)
    orc.prefill(pr, cfg.N)
    _iteration(cfg, eng, orc, 7, True)
    assert eng.device_status() == 0
    eng.close()


def test_sampling_needs_chain_drafts():
    from paper_2408_08146_b200 import KoalaError
    eng, _, _ = make_pair(TINY_EAGLE)                      # topk = 2: not a chain
    with pytest.raises(KoalaError) as e:
        eng.koala_set_sampling(torch.zeros(1, 4, device=DEV))
    assert e.value.code == 1
    eng.close()
