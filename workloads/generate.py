"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA library's callers.

Nothing here is part of the method: this module only produces *data* (weights, prompts,
KV contents, forced acceptance lengths, a static tree topology).  Every value is a pure
function of (seed, tensor id, element index) through a counter-based integer hash, so the
same tensors come out on a CPU and on a GPU and no generator state is carried between calls.

Value recipe: two 32-bit hashes -> two uniforms in (0, 1) -> Box-Muller in float64 ->
scale -> cast (round-to-nearest-even for bf16).
"""
from __future__ import annotations

import math
import zlib
from typing import Callable, Dict, List, Sequence

import numpy as np
import torch

from .configs import BF16, EAGLE, FP32, MEDUSA, KoalaConfig

_M32 = 0xFFFFFFFF


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Integer finaliser (the public-domain 'lowbias32' constants) on uint32 values held in int64."""
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def tensor_id(name: str) -> int:
    return zlib.crc32(name.encode()) & _M32


def _key(seed: int, tid: int, stream: int) -> int:
    return _mix32_int(_mix32_int(_mix32_int(seed) ^ tid) ^ (0x9E3779B9 * (stream + 1) & _M32))


def hashed_u32(seed: int, tid: int, stream: int, start: int, count: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix32(idx ^ _key(seed, tid, stream))


def uniform_ints(seed: int, name: str, count: int, lo: int, hi: int) -> np.ndarray:
    """count integers uniform in [lo, hi) (modulo bias < 2^-17 for the ranges used here)."""
    u = hashed_u32(seed, tensor_id(name), 0, 0, count, "cpu")
    return (lo + (u % (hi - lo))).numpy().astype(np.int32)


def normal_f64(seed: int, name: str, numel: int, device, chunk: int = 1 << 24) -> torch.Tensor:
    tid = tensor_id(name)
    out = torch.empty(numel, dtype=torch.float64, device=device)
    for s in range(0, numel, chunk):
        c = min(chunk, numel - s)
        u1 = (hashed_u32(seed, tid, 0, s, c, device).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        u2 = (hashed_u32(seed, tid, 1, s, c, device).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        out[s:s + c] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return out


def normal_tensor(seed: int, name: str, shape: Sequence[int], std: float, mean: float,
                  dtype: torch.dtype, device) -> torch.Tensor:
    n = int(np.prod(shape))
    t = normal_f64(seed, name, n, device)
    t.mul_(std).add_(mean)
    return t.to(dtype).reshape(*shape)


def torch_dtype(cfg: KoalaConfig) -> torch.dtype:
    return torch.float32 if cfg.dtype == FP32 else torch.bfloat16


LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def layer_shapes(cfg: KoalaConfig) -> Dict[str, tuple]:
    H, F = cfg.H, cfg.F
    return {"attn_norm": (H,), "wq": (H, H), "wk": (H, H), "wv": (H, H), "wo": (H, H),
            "ffn_norm": (H,), "w_gate": (F, H), "w_up": (F, H), "w_down": (H, F)}


def weight_shapes(cfg: KoalaConfig) -> Dict[str, tuple]:
    """Name -> shape of every tensor, row-major [out][in]."""
    H, V = cfg.H, cfg.V
    shapes: Dict[str, tuple] = {"embed": (V, H), "lm_head": (V, H), "final_norm": (H,)}
    for l in range(cfg.L):
        for t, s in layer_shapes(cfg).items():
            shapes[f"layers.{l}.{t}"] = s
    if cfg.head_kind == EAGLE:
        shapes["fc_w"] = (H, 2 * H)
        shapes["fc_b"] = (H,)
        for j in range(cfg.K):
            for t, s in layer_shapes(cfg).items():
                shapes[f"draft.{j}.{t}"] = s
    else:
        for i in range(cfg.n_medusa_heads):
            for j in range(cfg.K):
                shapes[f"medusa.{i}.{j}.w"] = (H, H)
                shapes[f"medusa.{i}.{j}.b"] = (H,)
            if cfg.medusa_own_lm:
                shapes[f"medusa.{i}.lm"] = (V, H)
    return shapes


class WeightStore:
    """All tensors of one configuration: N(0, 0.02) matrices and biases, norm gains 1 + N(0, 0.02).

    Tensors live on ``device`` in the configuration's storage dtype.  ``host(name)`` hands the
    values to a CPU consumer as a numpy array of the requested float type (exact upcast).
    """

    def __init__(self, cfg: KoalaConfig, device="cpu", std: float = 0.02):
        self.cfg = cfg
        self.device = torch.device(device)
        self.tensors: Dict[str, torch.Tensor] = {}
        dt = torch_dtype(cfg)
        for name, shape in weight_shapes(cfg).items():
            mean = 1.0 if name.endswith("norm") else 0.0
            self.tensors[name] = normal_tensor(cfg.seed, name, shape, std, mean, dt, self.device)

    def __getitem__(self, name: str) -> torch.Tensor:
        return self.tensors[name]

    def to(self, device) -> "WeightStore":
        """Moves every tensor (plain copies; the values were generated where the store was built)."""
        self.device = torch.device(device)
        self.tensors = {n: t.to(self.device) for n, t in self.tensors.items()}
        return self

    def host(self, name: str, dtype=np.float64) -> np.ndarray:
        t = self.tensors[name]
        if dtype == np.float64:
            return t.detach().to("cpu").to(torch.float64).numpy()
        return t.detach().to("cpu").to(torch.float32).numpy().astype(dtype, copy=False)

    def host_getter(self, dtype=np.float64) -> Callable[[str], np.ndarray]:
        return lambda name: self.host(name, dtype)

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.tensors.values())


def prompt_lengths(cfg: KoalaConfig) -> np.ndarray:
    if cfg.prompt_len_min > 0:
        return uniform_ints(1000 + cfg.seed, "prompt_len", cfg.B, cfg.prompt_len_min, cfg.prompt_len + 1)
    return np.full(cfg.B, cfg.prompt_len, dtype=np.int32)


def prompts(cfg: KoalaConfig) -> List[np.ndarray]:
    """One array of uniform-random token ids per sequence."""
    lens = prompt_lengths(cfg)
    return [uniform_ints(1000 + cfg.seed, f"prompt.{b}", int(lens[b]), 0, cfg.V) for b in range(cfg.B)]


def forced_lengths(seed: int, count: int, lam: float = 3.0, lo: int = 1, hi: int = 6) -> np.ndarray:
    """Accepted lengths (bonus token included) drawn from Poisson(lam) clipped to [lo, hi]."""
    rng = np.random.default_rng(seed)
    return np.clip(rng.poisson(lam, size=count), lo, hi).astype(np.int32)


def clipped_poisson_mean(lam: float = 3.0, lo: int = 1, hi: int = 6) -> float:
    total, p = 0.0, math.exp(-lam)
    for i in range(0, 120):
        total += min(max(i, lo), hi) * p
        p *= lam / (i + 1)
    return total


def random_kv(cfg: KoalaConfig, name: str, n_layers: int, device, std: float = 1.0) -> torch.Tensor:
    """Synthetic cache contents [n_layers][B][n_heads][S_max][head_dim] in the storage dtype."""
    shape = (n_layers, cfg.B, cfg.n_heads, cfg.S_max, cfg.head_dim)
    return normal_tensor(2000 + cfg.seed, name, shape, std, 0.0, torch_dtype(cfg), device)


def random_hidden(cfg: KoalaConfig, name: str, rows: int, device, dtype=torch.float32) -> torch.Tensor:
    return normal_tensor(3000 + cfg.seed, name, (rows, cfg.H), 1.0, 0.0, dtype, device)


# Chain-draft acceptance rates of the single-layer Medusa head on the 7B target (the paper's
# Table 1, rows 1-alpha / 2-alpha / 3-alpha); the fourth value is an extrapolation.
MEDUSA_ALPHA = (0.57, 0.40, 0.31, 0.25)


def medusa_static_tree(n_nodes: int = 64, depth: int = 4, width: int = 10,
                       alpha: Sequence[float] = MEDUSA_ALPHA, decay: float = 1.5):
    """Static candidate-tree topology: top-``width`` at depth 1, thinning with depth.

    Every rank path (r_1..r_d), d <= depth, r_i < width, gets the weight
    (alpha_1 .. alpha_d) * ((1+r_1) .. (1+r_d)) ** -decay; the n_nodes-1 heaviest paths are kept
    (ties: shallower first, then lexicographic).  Returns (parent, level, rank) int32 arrays with
    node 0 the root and nodes ordered by (level, path), so parents precede children.
    """
    cands = []

    def rec(path, prod_a, prod_r):
        d = len(path)
        if d:
            cands.append((-(prod_a * float(prod_r) ** (-decay)), d, tuple(path)))
        if d == depth:
            return
        for r in range(width):
            rec(path + [r], prod_a * alpha[d], prod_r * (1 + r))

    rec([], 1.0, 1)
    cands.sort()
    kept = sorted((c[1], c[2]) for c in cands[: n_nodes - 1])
    index = {(): 0}
    parent, level, rank = [-1], [0], [0]
    for d, path in kept:
        index[path] = len(parent)
        parent.append(index[path[:-1]])
        level.append(d)
        rank.append(path[-1])
    return (np.asarray(parent, np.int32), np.asarray(level, np.int32), np.asarray(rank, np.int32))


def chain_tree(tokens: Sequence[int]):
    """A chain (every node has one child): (tok, parent) arrays."""
    n = len(tokens)
    return np.asarray(tokens, np.int32), np.arange(-1, n - 1, dtype=np.int32)
