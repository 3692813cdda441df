"""Edge cases of the CUDA path against the oracle: degenerate trees, maximum tree size, a head
without layers, long contexts that span many key tiles and several key chunks, capacity and
malformed-input reporting, and the call-order rules."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle.koala_oracle import KoalaOracle, round_to_bf16
from paper_2408_08146_b200 import Koala, KoalaError
from tests.harness import kv_to_oracle, make_pair, tok_list
from tests.helpers import HostWeights
from tests.parity import assert_close, check_argmax
from workloads import T7_EAGLE, TINY_EAGLE, reduced
from workloads.generate import prompts, random_kv, uniform_ints

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _tree_arrays(eng, toks, parents):
    cfg = eng.cfg
    n = len(toks[0])
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)
    return to(toks), to(parents), to(np.full(cfg.B, n)), n


def test_single_node_tree_is_plain_autoregressive_decoding():
    cfg = TINY_EAGLE.with_(N=1, D=1, S_max=128)
    eng, orc, _ = make_pair(cfg)
    pr = prompts(cfg)
    # one token per call: 64 single-node chains, forced acceptance of 1 = the node itself
    for t in range(cfg.prompt_len):
        tree = _tree_arrays(eng, [[int(pr[0][t])]], [[-1]])
        eng.koala_verify(tree)
        eng.koala_accept(tree[2])
    orc.prefill(pr, 1)
    out = []
    for _ in range(6):
        root = eng.buffers()["root_tok"].cpu().numpy().reshape(1, 1)
        eng.koala_verify(_tree_arrays(eng, root, [[-1]]))
        tk, ln = tok_list(*eng.koala_accept(None))
        assert ln == [1]
        out += tk[0]
    assert out == orc.ar_greedy(6)[0]
    assert eng.device_status() == 0
    eng.close()


def test_maximum_tree_of_128_nodes_chain_and_bushy():
    cfg = TINY_EAGLE.with_(N=128, D=4, topk=2, S_max=400, prompt_len=128)
    eng, orc, _ = make_pair(cfg)
    pr = prompts(cfg)
    eng.prefill(pr, 128)                     # one chain of 128 nodes: every mask bit in use
    orc.prefill(pr, 128)
    assert eng.seq_len.cpu().tolist() == orc.seq_len == [128]
    for l in range(cfg.L):
        assert_close(kv_to_oracle(eng.target_k, l, 0, np.float64)[:128], orc.target_k[l][0][:128], cfg.dtype, "K")
    # a bushy 128-node caller tree on top of it
    n = 128
    par = [-1] + [int(p) for p in (uniform_ints(5, "edge.par", n - 1, 0, 1 << 20) % np.arange(1, n))]
    par = [-1 if u == 0 else min(par[u], u - 1) for u in range(n)]
    tok = uniform_ints(5, "edge.tok", n, 0, cfg.V)
    tok[0] = orc.root_tok[0]
    eng.koala_verify(_tree_arrays(eng, [tok], [par]))
    orc.verify([(tok, np.asarray(par))])
    b = eng.buffers()
    assert_close(b["verify_logits"][:n].cpu().numpy(), orc.verify_logits[0], cfg.dtype, "128-node tree logits")
    check_argmax(b["verify_tgt"][:n].cpu().numpy(), orc.verify_logits[0], "128-node tree arg-max")
    got = tok_list(*eng.koala_accept(None))
    ref = orc.accept()
    assert list(got[0]) == list(ref[0]) and list(got[1]) == list(ref[1])
    assert eng.device_status() == 0
    eng.close()


def test_eagle_head_without_layers():
    cfg = TINY_EAGLE.with_(K=0, S_max=160)
    eng, orc, _ = make_pair(cfg)
    pr = prompts(cfg)
    eng.prefill(pr, 15)
    orc.prefill(pr, 15)
    for _ in range(2):
        got = tok_list(*eng.step())
        ref = orc.step()
        assert list(got[0]) == ref[0] and list(got[1]) == ref[1]
        n = len(orc.tree_tok[0])
        assert eng.buffers()["tree_tok"][0, :n].cpu().tolist() == list(orc.tree_tok[0])
    assert eng.device_status() == 0
    eng.close()


@pytest.mark.parametrize("context", [1000, 3900])
def test_long_context_many_key_tiles_and_chunks(context):
    """bf16, head_dim 128, one 7B-shaped layer: the attention kernel walks dozens of key tiles and,
    at the longer context, several key chunks merged by the second kernel."""
    cfg = reduced(T7_EAGLE, 1, K=1, N=60, S_max=4096, prompt_len=context)
    eng, orc, _ = make_pair(cfg, oracle_dtype=np.float32, cache_host=False)
    eng.target_k.copy_(random_kv(cfg, "target_k", cfg.L, DEV))
    eng.target_v.copy_(random_kv(cfg, "target_v", cfg.L, DEV))
    orc.target_k[0][0][...] = kv_to_oracle(eng.target_k, 0, 0, np.float32)
    orc.target_v[0][0][...] = kv_to_oracle(eng.target_v, 0, 0, np.float32)
    eng.seq_len.fill_(context)
    orc.seq_len[0] = context
    n = cfg.N
    par = [-1] + [max(0, u - 1 - (u * 7) % min(u, 5)) for u in range(1, n)]
    tok = uniform_ints(9, "edge.long", n, 0, cfg.V)
    eng.koala_verify(_tree_arrays(eng, [tok], [par]))
    orc.verify([(tok, np.asarray(par))])
    b = eng.buffers()
    assert_close(b["verify_hid"][:n].cpu().numpy(), orc.verify_hid[0], cfg.dtype, f"hidden at context {context}")
    assert_close(b["verify_logits"][:n].cpu().numpy(), orc.verify_logits[0], cfg.dtype, f"logits at context {context}")
    assert eng.device_status() == 0
    eng.close()


@pytest.mark.parametrize("N,B,n_heads,context,S_max", [
    (128, 1, 32, 1000, 4096),    # more than 64 rows: every row warp owns its rows; 4 key chunks
    (100, 2, 32, 700, 1024),     # ragged row count above 64, 2 chunks, two sequences
    (20, 1, 32, 300, 512),       # fewer than 32 rows: one row group, duplicated
    (40, 8, 32, 200, 512),       # more CTAs than SMs: a single chunk, no cluster
    (60, 1, 8, 3000, 4096),      # few heads: 8 key chunks per head
    (33, 1, 32, 64, 256),        # a short context: one tile per chunk
    (33, 1, 32, 20, 1024),       # one key tile, four key chunks: three CTAs of a cluster have no tile and still merge and store their dims
    (60, 1, 8, 10, 4096),        # two key tiles, eight key chunks
])
def test_tensor_core_attention_shapes(N, B, n_heads, context, S_max):
    """One bf16 layer with head_dim 128 at row counts, batch sizes and chunk counts that select
    every variant of the tcgen05 attention kernel; the tree sits on top of a random cache."""
    _attention_case(N, B, n_heads, context, S_max)


@pytest.mark.parametrize("N,B,n_heads,context,S_max", [
    (60, 1, 32, 500, 1024),      # tcgen05 kernel, duplicated rows; the last key tile is partial
    (100, 2, 32, 700, 1024),     # tcgen05 kernel, more than 64 rows
    (8, 1, 32, 300, 512),        # fewer than 16 rows: the mma.sync kernel
])
def test_unwritten_cache_slots_may_hold_nan(N, B, n_heads, context, S_max):
    """Only the slots below seq_len (and the tree's own) ever hold data the caller or the library
    wrote; everything beyond may be uninitialised memory.  The slots from S + N on are filled with
    NaN bit patterns here (plain data, nothing faults) and the result must not change."""
    _attention_case(N, B, n_heads, context, S_max, poison=True)


@pytest.mark.parametrize("N,B,n_heads,context,S_max", [
    (60, 1, 32, 1000, 2048),     # duplicated rows, 4 key chunks of several tiles each
    (128, 1, 32, 1500, 4096),    # every row warp owns its rows
])
def test_scores_that_grow_along_the_context(N, B, n_heads, context, S_max):
    """Keys whose magnitude grows eightfold from the first to the last cached position: the row
    maxima rise by far more than 2^8 from tile to tile, so the running output, which the tcgen05
    kernel keeps in tensor memory relative to a lazily raised reference maximum, is rescaled in place
    several times."""
    _attention_case(N, B, n_heads, context, S_max, growing=True)


def _attention_case(N, B, n_heads, context, S_max, poison=False, growing=False):
    H = n_heads * 128
    cfg = reduced(T7_EAGLE, 1, K=1, N=N, B=B, H=H, n_heads=n_heads, F=2 * H, V=2048, D=min(5, N - 1),
                  S_max=S_max, prompt_len=context)
    eng, orc, _ = make_pair(cfg, oracle_dtype=np.float32, cache_host=False)
    eng.target_k.copy_(random_kv(cfg, "target_k", cfg.L, DEV))
    eng.target_v.copy_(random_kv(cfg, "target_v", cfg.L, DEV))
    if growing:
        ramp = 1.0 + 7.0 * torch.arange(S_max, device=DEV, dtype=torch.float32) / context
        eng.target_k.copy_((eng.target_k.float() * ramp.view(1, 1, 1, S_max, 1)).to(eng.target_k.dtype))
    lens = [context - 13 * b for b in range(B)]
    for b in range(B):
        orc.target_k[0][b][...] = kv_to_oracle(eng.target_k, 0, b, np.float32)
        orc.target_v[0][b][...] = kv_to_oracle(eng.target_v, 0, b, np.float32)
        orc.seq_len[b] = lens[b]
    eng.seq_len.copy_(torch.tensor(lens, dtype=torch.int32))
    if poison:
        for b in range(B):
            eng.target_k[:, b, :, lens[b] + N:, :] = float("nan")
            eng.target_v[:, b, :, lens[b] + N:, :] = float("nan")
    par = [-1] + [max(0, u - 1 - (u * 7) % min(u, 5)) for u in range(1, N)]
    toks = [uniform_ints(11 + b, "edge.shapes", N, 0, cfg.V) for b in range(B)]
    eng.koala_verify(_tree_arrays(eng, toks, [par] * B))
    orc.verify([(toks[b], np.asarray(par)) for b in range(B)])
    bufs = eng.buffers()
    for b in range(B):
        assert_close(bufs["verify_hid"][b * N:(b + 1) * N].cpu().numpy(), orc.verify_hid[b], cfg.dtype,
                     f"hidden, sequence {b}")
    assert eng.device_status() == 0
    eng.close()


def test_capacity_and_malformed_trees_are_reported_not_executed():
    cfg = TINY_EAGLE.with_(S_max=80)                    # the 64-token prompt fits, prompt + tree does not
    eng, orc, _ = make_pair(cfg)
    pr = prompts(cfg)
    eng.prefill(pr, 15)
    assert eng.device_status() == 0
    eng.seq_len.fill_(70)                               # 70 + 15 > 80
    k_before = eng.target_k.clone()
    eng.koala_verify(_tree_arrays(eng, [[1] * 15], [list(range(-1, 14))]))
    assert eng.device_status() == 3                     # KOALA_E_CAPACITY, from the plan kernel
    assert torch.equal(k_before, eng.target_k)          # nothing was written past the capacity
    eng.close()
    eng, _, _ = make_pair(TINY_EAGLE)
    eng.koala_verify(_tree_arrays(eng, [[1, 2, 3]], [[-1, 2, 0]]))     # parent index not below the child
    assert eng.device_status() == 1                     # KOALA_E_INVALID
    eng.close()


def test_call_order_and_argument_errors():
    eng, _, _ = make_pair(TINY_EAGLE)
    with pytest.raises(KoalaError) as e:
        eng.koala_expand_tree(0)                        # nothing drafted
    assert e.value.code == 4
    with pytest.raises(KoalaError) as e:
        eng.koala_draft(1)                              # pass 1 before pass 0
    assert e.value.code == 4
    with pytest.raises(KoalaError) as e:
        eng.koala_draft(99)
    assert e.value.code == 1
    with pytest.raises(KoalaError) as e:
        eng.koala_verify(None)                          # no drafted tree
    assert e.value.code == 4
    with pytest.raises(KoalaError) as e:
        eng.koala_accept(None)                          # nothing verified
    assert e.value.code == 4
    tok = torch.zeros(1, 16, dtype=torch.int32, device=DEV)
    with pytest.raises(KoalaError) as e:
        eng.koala_verify((tok, tok, torch.ones(1, dtype=torch.int32, device=DEV), 16))   # n_max > N
    assert e.value.code == 1
    eng.close()


def test_position_wise_acceptance_counters_match_the_oracle():
    """n-alpha counters (Section 4.1, metrics): chains whose first m tokens are the target's own
    greedy continuation, then free-running iterations with the head's real trees; the device
    counters equal the oracle's and, for the planted part, the tally made here from (m, d)."""
    cfg = TINY_EAGLE.with_(S_max=256)
    eng, orc, store = make_pair(cfg)
    pr = prompts(cfg)
    eng.prefill(pr, 15)
    orc.prefill(pr, 15)
    truth_src = KoalaOracle(cfg, HostWeights(store, np.float64))
    truth_src.prefill(pr, 64)
    truth = truth_src.ar_greedy(80)[0]
    eng.koala_accept_stats(1, reset=True)
    orc.reset_alpha()
    hits, trials = [0] * cfg.N, [0] * cfg.N
    emitted = 0
    for it in range(10):
        d = 1 + (it * 3) % 5
        m = (it * 7) % (d + 1)
        tok = [int(orc.root_tok[0])]
        for i in range(d):
            t = int(truth[emitted + i])
            tok.append(t if i < m else (t + 1 + 13 * it) % cfg.V)
        par = list(range(-1, d))
        eng.koala_verify(_tree_arrays(eng, [tok], [par]))
        orc.verify([(np.asarray(tok), np.asarray(par))])
        got = tok_list(*eng.koala_accept(None))
        ref = orc.accept()
        assert list(got[1]) == list(ref[1]) == [m + 1] and list(got[0][0]) == list(ref[0][0])
        emitted += m + 1
        for n in range(1, d + 1):
            trials[n - 1] += n <= m + 1
            hits[n - 1] += n <= m
    g_hits, g_trials = eng.koala_accept_stats(cfg.N)
    assert g_hits == hits == orc.alpha_hits[:cfg.N] and g_trials == trials == orc.alpha_trials[:cfg.N]
    for _ in range(4):                                   # the head's own trees
        got = tok_list(*eng.step())
        ref = orc.step()
        assert list(got[0]) == ref[0] and list(got[1]) == ref[1]
    g_hits, g_trials = eng.koala_accept_stats(cfg.N, reset=True)
    assert g_hits == orc.alpha_hits[:cfg.N] and g_trials == orc.alpha_trials[:cfg.N]
    assert eng.koala_accept_stats(cfg.N) == ([0] * cfg.N, [0] * cfg.N)
    assert eng.device_status() == 0
    eng.close()


def test_whole_iterations_repeat_bit_for_bit():
    """Two engines on the same weights, prompts ingested in chunks (the first chunks have fewer key
    tiles than key chunks), several forced iterations: trees, target tokens and accepted tokens must
    be identical."""
    from workloads import T7_EAGLE, reduced
    from workloads.generate import WeightStore
    from paper_2408_08146_b200 import Koala
    cfg = reduced(T7_EAGLE, 2, K=1, S_max=768, prompt_len=300)
    store = WeightStore(cfg, DEV)
    forced = torch.tensor([[3], [1], [5], [2]], dtype=torch.int32, device=DEV)
    runs = []
    for _ in range(2):
        eng = Koala(cfg, store.tensors)
        eng.prefill(prompts(cfg), 64)
        rec = [eng.buffers()["root_tok"].cpu().numpy().copy()]
        for i in range(forced.shape[0]):
            toks, lens = eng.step(forced[i])
            torch.cuda.synchronize()
            b = eng.buffers()
            n = int(b["tree_n"][0].item())
            rec += [lens.cpu().numpy().copy(), toks[0, :int(lens[0].item())].cpu().numpy().copy(),
                    b["tree_tok"][0, :n].cpu().numpy().copy(), b["verify_tgt"][:n].cpu().numpy().copy()]
        assert eng.device_status() == 0
        eng.close()
        runs.append(rec)
    for a, c in zip(*runs):
        assert np.array_equal(a, c)
