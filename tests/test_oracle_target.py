"""Pins of the oracle's target forward (decoder stack, tree mask, chain / single-node cases)."""
import itertools

import numpy as np
import pytest
import torch

from oracle.koala_oracle import KoalaOracle, ancestor_matrix, tree_levels
from tests.helpers import HostWeights
from workloads import TINY_EAGLE
from workloads.generate import WeightStore, prompts

CFG = TINY_EAGLE.with_(S_max=96)


@pytest.fixture(scope="module")
def hw():
    return HostWeights(WeightStore(CFG))


def _full_forward(hw, tokens):
    """Logits of a plain causal forward over `tokens` from an empty cache (chain tree)."""
    o = KoalaOracle(CFG, hw)
    logits, hid = o.target_forward(0, np.asarray(tokens), np.arange(-1, len(tokens) - 1))
    return logits, hid, o


def test_decoder_stack_matches_transformers_llama(hw):
    """Library pin: the same weights loaded into `transformers`' Llama give the same logits.

    Covers RMSNorm, the half-split RoPE convention with base 10000, scaled causal softmax
    attention, SwiGLU, the residual wiring, the final norm and the LM head.
    """
    from transformers import LlamaConfig, LlamaForCausalLM
    c = CFG
    hf_cfg = LlamaConfig(hidden_size=c.H, intermediate_size=c.F, num_hidden_layers=c.L,
                         num_attention_heads=c.n_heads, num_key_value_heads=c.n_heads,
                         vocab_size=c.V, rms_norm_eps=c.rms_eps, rope_theta=c.rope_base,
                         max_position_embeddings=512, tie_word_embeddings=False,
                         attention_bias=False, mlp_bias=False, head_dim=c.head_dim,
                         attn_implementation="eager")
    model = LlamaForCausalLM(hf_cfg).double().eval()
    sd = {"model.embed_tokens.weight": hw("embed"), "model.norm.weight": hw("final_norm"),
          "lm_head.weight": hw("lm_head")}
    names = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
             "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    for l in range(c.L):
        for ours, theirs in names.items():
            sd[f"model.layers.{l}.{theirs}.weight"] = hw(f"layers.{l}.{ours}")
    missing, unexpected = model.load_state_dict({k: torch.from_numpy(np.array(v)) for k, v in sd.items()},
                                                strict=False)
    assert not [m for m in missing if "rotary" not in m] and not unexpected
    toks = prompts(CFG)[0][:40]
    with torch.no_grad():
        ref = model(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    ours, _, _ = _full_forward(hw, toks)
    # the library evaluates its rotary tables in float32 whatever the model dtype, which leaves
    # ~1e-7 of difference; a wrong convention anywhere shows up at the scale of the logits (~1)
    assert np.max(np.abs(ours - ref)) < 1e-5
    assert np.std(ref) > 0.1


def test_tree_verify_equals_per_path_causal_forward(hw):
    """Brute force: every node's logits equal those of a causal forward over prompt + its path."""
    prompt = prompts(CFG)[0][:20]
    o = KoalaOracle(CFG, hw)
    o.prefill([prompt], 8)
    assert o.seq_len == [20]
    #            0   1  2  3  4  5  6  7  8  9
    parent = [-1, 0, 0, 1, 1, 2, 3, 3, 5, 8]
    tok = np.asarray([7, 100, 200, 300, 301, 17, 900, 901, 5, 1023])
    logits, hid = o.target_forward(0, tok, np.asarray(parent))
    vis = ancestor_matrix(parent)
    for u in range(len(parent)):
        path = [v for v in range(len(parent)) if vis[u, v]]
        seq = list(prompt) + [int(tok[v]) for v in path]
        ref, ref_hid, _ = _full_forward(hw, seq)
        assert np.max(np.abs(ref[-1] - logits[u])) < 1e-9
        assert np.max(np.abs(ref_hid[-1] - hid[u])) < 1e-9


def test_chain_chunks_equal_one_shot_prefill_and_single_node_decode(hw):
    prompt = prompts(CFG)[0][:33]
    ref, _, o_ref = _full_forward(hw, prompt)
    o = KoalaOracle(CFG, hw)
    o.prefill([prompt[:32]], 5)                    # ragged chunking
    for l in range(CFG.L):
        assert np.max(np.abs(o.target_k[l][0][:32] - o_ref.target_k[l][0][:32])) < 1e-10
        assert np.max(np.abs(o.target_v[l][0][:32] - o_ref.target_v[l][0][:32])) < 1e-10
    # N = 1: one more token as a single-node tree reproduces the last row of the full forward
    logits, _ = o.target_forward(0, prompt[32:33], np.asarray([-1]))
    assert np.max(np.abs(logits[0] - ref[32])) < 1e-9
    # and the prefill's bonus token is the greedy token after the 32-token prefix
    assert o.root_tok[0] == int(np.argmax(ref[31]))


def test_tree_helpers():
    parent = [-1, 0, 0, 1, 3]
    assert list(tree_levels(parent)) == [0, 1, 1, 2, 3]
    vis = ancestor_matrix(parent)
    assert vis[4].tolist() == [True, True, False, True, True]
    assert vis[2].tolist() == [True, False, True, False, False]
    with pytest.raises(AssertionError):
        tree_levels([-1, 2, 0])


def test_cache_storage_rounding_is_applied_to_rotated_keys_and_values_only(hw):
    """Where the oracle rounds for a bf16 cache (the paper states no precision, Section 4.1; the
    reading is: a key / value is rounded when it is written to the cache, after the rotary
    embedding, and nothing else is rounded).

    (1) A recording identity in place of the rounding: the run is bit-equal to the run without it,
    it is called exactly twice per layer and forward, and what it is handed is exactly what the
    un-rounded run stores (the rotated keys, the values) - so queries never pass through it and a
    rounding placed before the rotation would be handed something else.
    (2) With the real rounding, layer 0 (whose inputs do not depend on any cache) stores exactly
    the rounded values of the un-rounded run, bit for bit, and later layers see a different cache.
    """
    from oracle.koala_oracle import round_to_bf16
    toks = prompts(CFG)[0][:24]
    par = np.arange(-1, len(toks) - 1)
    plain = KoalaOracle(CFG, hw, dtype=np.float32)
    ref_logits, _ = plain.target_forward(0, toks, par)

    seen = []

    def recording_identity(a):
        seen.append(np.array(a, copy=True))
        return a

    rec = KoalaOracle(CFG, hw, dtype=np.float32, kv_round=recording_identity)
    logits, _ = rec.target_forward(0, toks, par)
    assert np.array_equal(logits, ref_logits)
    assert len(seen) == 2 * CFG.L
    n = len(toks)
    for l in range(CFG.L):
        assert seen[2 * l].shape == seen[2 * l + 1].shape == (n, CFG.n_heads, CFG.head_dim)
        assert np.array_equal(seen[2 * l], plain.target_k[l][0][:n])        # rotated keys
        assert np.array_equal(seen[2 * l + 1], plain.target_v[l][0][:n])    # values

    rounded = KoalaOracle(CFG, hw, dtype=np.float32, kv_round=round_to_bf16)
    r_logits, _ = rounded.target_forward(0, toks, par)
    k0, v0 = rounded.target_k[0][0][:n], rounded.target_v[0][0][:n]
    assert np.array_equal(k0.view(np.uint32), round_to_bf16(plain.target_k[0][0][:n]).view(np.uint32))
    assert np.array_equal(v0.view(np.uint32), round_to_bf16(plain.target_v[0][0][:n]).view(np.uint32))
    assert (k0.view(np.uint32) & 0xFFFF == 0).all() and (v0.view(np.uint32) & 0xFFFF == 0).all()
    # rounding the keys before rotating them gives other bits: the check above can tell the two apart
    from oracle.koala_oracle import rmsnorm, rope
    x0 = hw("embed").astype(np.float32)[np.asarray(toks, dtype=np.int64)]
    h0 = rmsnorm(x0, hw("layers.0.attn_norm").astype(np.float32), CFG.rms_eps)
    k_pre = (h0 @ hw("layers.0.wk").astype(np.float32).T).reshape(n, CFG.n_heads, CFG.head_dim)
    slip = rope(round_to_bf16(k_pre), np.arange(n), CFG.rope_base)
    assert not np.array_equal(np.asarray(slip, np.float32).view(np.uint32), k0.view(np.uint32))
    # the rounded cache changes the result, but only at the scale of bf16 rounding
    d = np.abs(r_logits - ref_logits).max()
    assert 0 < d < 5e-2
