"""Workload descriptions for the draft-then-verify step (shapes only, no arithmetic).

Symbols follow the speculative-decoding statement of the paper (Section 2.2) and its
multi-layer draft heads (Section 3.1): a target LLM with ``L`` decoder layers, a draft head
with ``K`` layers, ``D`` draft levels, top-``k`` expansion and a candidate tree of ``N`` nodes
(root included).
"""
from __future__ import annotations

from dataclasses import dataclass, replace, asdict

EAGLE = 0
MEDUSA = 1

FP32 = 0
BF16 = 1


@dataclass(frozen=True)
class KoalaConfig:
    name: str
    dtype: int            # FP32 or BF16 (storage of weights / KV; accumulation is fp32)
    head_kind: int        # EAGLE or MEDUSA
    L: int                # target decoder layers
    H: int                # hidden size
    n_heads: int
    head_dim: int
    F: int                # SwiGLU width
    V: int                # vocabulary
    K: int                # draft-head layers (Section 3.1)
    D: int                # draft levels below the root
    topk: int             # expansion width k
    N: int                # tree nodes including the root
    B: int = 1            # sequences per step
    S_max: int = 256      # KV capacity per sequence
    n_medusa_heads: int = 0
    medusa_own_lm: bool = False   # Medusa-style heads each end in a Linear of their own instead of the shared LM head
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    prompt_len: int = 64  # context length of the synthetic prompt (max, if ragged)
    prompt_len_min: int = 0   # >0: ragged prompt lengths uniform in [min, prompt_len]
    seed: int = 0

    def with_(self, **kw) -> "KoalaConfig":
        return replace(self, **kw)

    def to_dict(self) -> dict:
        return asdict(self)


# Tiny fp32 Llama-style target with a 2-layer EAGLE-style head: depth 4, top-2, 15 nodes.
TINY_EAGLE = KoalaConfig(
    name="tiny_eagle_fp32", dtype=FP32, head_kind=EAGLE, L=2, H=256, n_heads=4, head_dim=64,
    F=688, V=1024, K=2, D=4, topk=2, N=15, B=1, S_max=192, prompt_len=64, seed=0)

# Same tiny target with Medusa-style heads (used by CPU tests of the non-autoregressive path).
TINY_MEDUSA = TINY_EAGLE.with_(name="tiny_medusa_fp32", head_kind=MEDUSA, K=2, D=3, topk=3,
                               N=12, n_medusa_heads=3, seed=5)

# 7B-shaped target, Medusa-style heads: 4 heads x K=2 residual blocks, static 64-node tree.
T7_MEDUSA = KoalaConfig(
    name="t7_medusa_bf16", dtype=BF16, head_kind=MEDUSA, L=32, H=4096, n_heads=32, head_dim=128,
    F=11008, V=32000, K=2, D=4, topk=10, N=64, B=1, S_max=1024, n_medusa_heads=4,
    prompt_len=512, seed=1)

# 7B-shaped target, EAGLE-style head with K decoder layers, dynamic tree depth 5 / top-10 / 60.
T7_EAGLE = KoalaConfig(
    name="t7_eagle_bf16", dtype=BF16, head_kind=EAGLE, L=32, H=4096, n_heads=32, head_dim=128,
    F=11008, V=32000, K=2, D=5, topk=10, N=60, B=1, S_max=1536, prompt_len=1024, seed=2)

# 13B-shaped target, batch 4 with ragged prompts, EAGLE-style head K=2, 64-node tree.
T13_EAGLE = KoalaConfig(
    name="t13_eagle_bf16", dtype=BF16, head_kind=EAGLE, L=40, H=5120, n_heads=40, head_dim=128,
    F=13824, V=32000, K=2, D=5, topk=10, N=64, B=4, S_max=2560, prompt_len=2048,
    prompt_len_min=512, seed=3)

# 33B-shaped target (hidden 6656 = 52 heads x 128, FFN 17920, 60 layers), EAGLE-style head; the
# paper expects larger K to pay off for larger targets (Section 4.2), so K is left to the caller.
T33_EAGLE = KoalaConfig(
    name="t33_eagle_bf16", dtype=BF16, head_kind=EAGLE, L=60, H=6656, n_heads=52, head_dim=128,
    F=17920, V=32000, K=2, D=5, topk=10, N=60, B=1, S_max=1536, prompt_len=1024, seed=7)

CONFIGS = [TINY_EAGLE, T7_MEDUSA, T7_EAGLE, T13_EAGLE]


def reduced(cfg: KoalaConfig, L: int, **kw) -> KoalaConfig:
    """Same per-layer shapes with fewer target layers (keeps every kernel's tile shapes)."""
    return cfg.with_(name=f"{cfg.name}_L{L}", L=L, **kw)
