"""Builds the CUDA engine and the oracle on the same seeded inputs (GPU tests only)."""
import numpy as np
import torch

from oracle.koala_oracle import KoalaOracle, round_to_bf16
from paper_2408_08146_b200 import Koala
from tests.helpers import HostWeights
from workloads.generate import WeightStore, medusa_static_tree

MEDUSA = 1


class StreamedWeights:
    """name -> host array straight from the device tensors (no host copy is kept)."""

    def __init__(self, store, dtype):
        self.store, self.dtype = store, dtype

    def __call__(self, name):
        return self.store.host(name, self.dtype)


def static_tree_for(cfg):
    if cfg.head_kind != MEDUSA:
        return None
    return medusa_static_tree(cfg.N, cfg.n_medusa_heads, cfg.topk)


def make_pair(cfg, flags=0, oracle_dtype=np.float64, cache_host=True):
    store = WeightStore(cfg, "cuda:0")
    st = static_tree_for(cfg)
    eng = Koala(cfg, store.tensors, static_tree=st, flags=flags)
    getter = HostWeights(store, oracle_dtype) if cache_host else StreamedWeights(store, oracle_dtype)
    orc = KoalaOracle(cfg, getter, dtype=oracle_dtype, static_tree=st,
                      kv_round=round_to_bf16 if cfg.dtype == 1 else None)
    return eng, orc, store


def kv_to_oracle(cache_t, l, b, dtype):
    """[L][B][nh][S_max][dh] device tensor -> the oracle's [S_max][nh][dh] array of one layer/sequence."""
    return cache_t[l, b].permute(1, 0, 2).to(torch.float32).cpu().numpy().astype(dtype)


def tok_list(out_tokens, out_len):
    t, n = out_tokens.cpu().numpy(), out_len.cpu().numpy()
    return [list(map(int, t[b, :n[b]])) for b in range(len(n))], list(map(int, n))
