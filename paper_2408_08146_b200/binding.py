"""Thin ctypes binding of libkoala.so: argument marshalling only.

Every step of the draft-then-verify iteration runs in the library's CUDA kernels; PyTorch is
used here for device memory, streams and copies.  There is no CPU fallback: if the library
cannot be built or loaded, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

from . import build as _build

KOALA_OK = 0
ERR_NAMES = {0: "KOALA_OK", 1: "KOALA_E_INVALID", 2: "KOALA_E_UNSUPPORTED", 3: "KOALA_E_CAPACITY",
             4: "KOALA_E_STATE", 5: "KOALA_E_CUDA", 6: "KOALA_E_TIMEOUT"}
KOALA_FP32, KOALA_BF16 = 0, 1
KOALA_EAGLE, KOALA_MEDUSA = 0, 1
KOALA_F_NO_TENSOR_CORES, KOALA_F_NO_PDL, KOALA_F_LAYER_KERNEL = 1, 2, 4
LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class KoalaError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {text}")
        self.code = code


class koala_config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("dtype", C.c_int32), ("head_kind", C.c_int32),
                ("L", C.c_int32), ("H", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("F", C.c_int32), ("V", C.c_int32), ("rms_eps", C.c_float), ("rope_base", C.c_float),
                ("K", C.c_int32), ("n_medusa_heads", C.c_int32), ("D", C.c_int32), ("topk", C.c_int32),
                ("N", C.c_int32), ("B", C.c_int32), ("S_max", C.c_int32), ("flags", C.c_uint32)]


class koala_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layer_w", C.POINTER(C.c_void_p)), ("fc_w", C.c_void_p), ("fc_b", C.c_void_p),
                ("draft_layer_w", C.POINTER(C.c_void_p)), ("res_w", C.POINTER(C.c_void_p)),
                ("res_b", C.POINTER(C.c_void_p)), ("medusa_lm", C.POINTER(C.c_void_p)),
                ("static_parent", C.POINTER(C.c_int32)),
                ("static_level", C.POINTER(C.c_int32)), ("static_rank", C.POINTER(C.c_int32))]


class koala_state(C.Structure):
    _fields_ = [("target_k", C.c_void_p), ("target_v", C.c_void_p), ("draft_k", C.c_void_p),
                ("draft_v", C.c_void_p), ("seq_len", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t)]


class koala_tree(C.Structure):
    _fields_ = [("tok", C.c_void_p), ("parent", C.c_void_p), ("n_nodes", C.c_void_p),
                ("stride", C.c_int32), ("n_max", C.c_int32)]


class koala_buffer_table(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "draft_logits", "draft_feat", "topk_tok", "topk_logp", "cand_tok", "cand_parent", "cand_score",
        "frontier", "tree_tok", "tree_parent", "tree_level", "tree_score", "tree_n", "verify_logits",
        "verify_hid", "verify_tgt", "root_tok", "pend_hid", "pend_tok", "n_pend", "acc_path")] + [
        ("pool", C.c_int32), ("draft_rows", C.c_int32)]


class koala_timing(C.Structure):
    _fields_ = [("ms", C.c_float * 3), ("bytes", C.c_uint64 * 3), ("launches", C.c_int32 * 3)]


_lib = None


def load_library(rebuild: bool = False) -> C.CDLL:
    """Builds (if stale) and loads libkoala.so; raises if that is not possible."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = os.environ.get("KOALA_LIBRARY") or _build.build(force=rebuild)   # an explicit library wins
    lib = C.CDLL(path)
    lib.koala_workspace_bytes.restype = C.c_size_t
    lib.koala_workspace_bytes.argtypes = [C.POINTER(koala_config)]
    lib.koala_init.restype = C.c_int
    lib.koala_init.argtypes = [C.POINTER(koala_config), C.POINTER(koala_weights), C.POINTER(koala_state),
                               C.c_void_p, C.POINTER(C.c_void_p)]
    lib.koala_draft.restype = C.c_int
    lib.koala_draft.argtypes = [C.c_void_p, C.c_int]
    lib.koala_expand_tree.restype = C.c_int
    lib.koala_expand_tree.argtypes = [C.c_void_p, C.c_int]
    lib.koala_verify.restype = C.c_int
    lib.koala_verify.argtypes = [C.c_void_p, C.POINTER(koala_tree)]
    lib.koala_set_sampling.restype = C.c_int
    lib.koala_set_sampling.argtypes = [C.c_void_p, C.c_void_p]
    lib.koala_accept_sampled.restype = C.c_int
    lib.koala_accept_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
    lib.koala_accept_stats.restype = C.c_int
    lib.koala_accept_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32]
    lib.koala_accept.restype = C.c_int
    lib.koala_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
    lib.koala_buffers.restype = C.c_int
    lib.koala_buffers.argtypes = [C.c_void_p, C.POINTER(koala_buffer_table)]
    lib.koala_set_option.restype = C.c_int
    lib.koala_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int]
    lib.koala_timing_read.restype = C.c_int
    lib.koala_timing_read.argtypes = [C.c_void_p, C.POINTER(koala_timing)]
    lib.koala_gemm_static_scratch_bytes.restype = C.c_size_t
    lib.koala_gemm_static_scratch_bytes.argtypes = []
    lib.koala_gemm_bf16_static.restype = C.c_int
    lib.koala_gemm_bf16_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                           C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    lib.koala_set_tuning.restype = None
    lib.koala_set_tuning.argtypes = [C.c_int, C.c_int]
    lib.koala_launch_count.restype = C.c_uint64
    lib.koala_launch_count.argtypes = []
    lib.koala_selftest_timeout.restype = C.c_int
    lib.koala_selftest_timeout.argtypes = [C.c_void_p, C.c_int]
    lib.koala_debug_check_guards.restype = C.c_int
    lib.koala_debug_check_guards.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.koala_poll.restype = C.c_int
    lib.koala_poll.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.koala_last_error.restype = C.c_char_p
    lib.koala_last_error.argtypes = [C.c_void_p]
    lib.koala_destroy.restype = None
    lib.koala_destroy.argtypes = [C.c_void_p]
    lib.koala_gemm_x_rows.restype = C.c_int
    lib.koala_gemm_x_rows.argtypes = [C.c_int, C.c_int]
    lib.koala_gemm_scratch_bytes.restype = C.c_size_t
    lib.koala_gemm_scratch_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
    lib.koala_gemm_bf16.restype = C.c_int
    lib.koala_gemm_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    _lib = lib
    return lib


def make_config(cfg, flags: int = 0) -> koala_config:
    """cfg: any object with the workload fields (L, H, n_heads, ..., S_max)."""
    return koala_config(C.sizeof(koala_config), int(cfg.dtype), int(cfg.head_kind), cfg.L, cfg.H,
                        cfg.n_heads, cfg.head_dim, cfg.F, cfg.V, cfg.rms_eps, cfg.rope_base, cfg.K,
                        cfg.n_medusa_heads, cfg.D, cfg.topk, cfg.N, cfg.B, cfg.S_max, flags)


def koala_workspace_bytes(cfg, flags: int = 0) -> int:
    c = make_config(cfg, flags)
    return int(load_library().koala_workspace_bytes(C.byref(c)))


def _ptr_array(tensors: Sequence[torch.Tensor]):
    arr = (C.c_void_p * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr()
    return arr


def _i32_array(values) -> "C.Array":
    v = np.ascontiguousarray(values, dtype=np.int32)
    arr = (C.c_int32 * len(v))()
    C.memmove(arr, v.ctypes.data, v.nbytes)
    return arr


def koala_gemm_bf16(x: torch.Tensor, w: torch.Tensor, use_tensor_cores: bool = True, split_k: int = 0,
                    status: Optional[torch.Tensor] = None, x_lo: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y[M][N] fp32 = (x [+ x_lo])[M][K] (bf16) @ w[N][K]^T (bf16) through the library's GEMM."""
    lib = load_library()
    M, K = x.shape
    N = w.shape[0]
    rows = int(lib.koala_gemm_x_rows(M, int(x_lo is not None)))             # whole token tiles
    xp = torch.zeros(rows, K, dtype=torch.bfloat16, device=x.device)
    xp[:M] = x
    xlp = None
    if x_lo is not None:
        xlp = torch.zeros(rows, K, dtype=torch.bfloat16, device=x.device)
        xlp[:M] = x_lo
    y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    nbytes = int(lib.koala_gemm_scratch_bytes(M, N, K))
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=x.device)
    st = torch.cuda.current_stream(x.device).cuda_stream
    rc = lib.koala_gemm_bf16(xp.data_ptr(), xlp.data_ptr() if xlp is not None else None, w.data_ptr(),
                             y.data_ptr(), N, M, N, K, scratch.data_ptr(),
                             nbytes, int(use_tensor_cores), split_k, st,
                             status.data_ptr() if status is not None else None)
    if rc != KOALA_OK:
        raise KoalaError(rc, "koala_gemm_bf16")
    # keep the operands alive until the stream has consumed them
    y._koala_keep = (xp, xlp, scratch, w)
    return y


class Koala:
    """Owns the device buffers of one context and forwards the five calls."""

    def __init__(self, cfg, weights: Dict[str, torch.Tensor], static_tree=None, flags: int = 0,
                 device: str = "cuda:0"):
        self.lib = load_library()
        self.cfg = cfg
        self.dev = torch.device(device)
        self.weights = weights
        self._ctx = C.c_void_p(None)
        dt = torch.float32 if cfg.dtype == KOALA_FP32 else torch.bfloat16
        for name, t in weights.items():
            if t.device != self.dev or t.dtype != dt or not t.is_contiguous():
                raise ValueError(f"weight {name} must be a contiguous {dt} tensor on {self.dev}")
        kv_shape = (cfg.L, cfg.B, cfg.n_heads, cfg.S_max, cfg.head_dim)
        self.target_k = torch.zeros(kv_shape, dtype=dt, device=self.dev)
        self.target_v = torch.zeros(kv_shape, dtype=dt, device=self.dev)
        eagle = cfg.head_kind == KOALA_EAGLE
        n_dkv = cfg.K if eagle else 0
        dkv_shape = (max(n_dkv, 1), cfg.B, cfg.n_heads, cfg.S_max, cfg.head_dim)
        self.draft_k = torch.zeros(dkv_shape, dtype=dt, device=self.dev)
        self.draft_v = torch.zeros(dkv_shape, dtype=dt, device=self.dev)
        self.seq_len = torch.zeros(cfg.B, dtype=torch.int32, device=self.dev)
        self._cfg_c = make_config(cfg, flags)
        nbytes = int(self.lib.koala_workspace_bytes(C.byref(self._cfg_c)))
        if nbytes == 0:
            raise KoalaError(1, "configuration rejected by koala_workspace_bytes")
        self.workspace = torch.zeros(nbytes + 256, dtype=torch.uint8, device=self.dev)
        self._ws_off = (-self.workspace.data_ptr()) % 256
        w = koala_weights()
        w.embed, w.lm_head, w.final_norm = (weights[n].data_ptr() for n in ("embed", "lm_head", "final_norm"))
        self._layer_arr = _ptr_array([weights[f"layers.{l}.{t}"] for l in range(cfg.L) for t in LAYER_TENSORS])
        w.layer_w = C.cast(self._layer_arr, C.POINTER(C.c_void_p))
        if eagle:
            w.fc_w, w.fc_b = weights["fc_w"].data_ptr(), weights["fc_b"].data_ptr()
            self._draft_arr = _ptr_array([weights[f"draft.{j}.{t}"] for j in range(cfg.K) for t in LAYER_TENSORS])
            w.draft_layer_w = C.cast(self._draft_arr, C.POINTER(C.c_void_p))
        else:
            hk = [(i, j) for i in range(cfg.n_medusa_heads) for j in range(cfg.K)]
            self._res_w = _ptr_array([weights[f"medusa.{i}.{j}.w"] for i, j in hk])
            self._res_b = _ptr_array([weights[f"medusa.{i}.{j}.b"] for i, j in hk])
            w.res_w = C.cast(self._res_w, C.POINTER(C.c_void_p))
            w.res_b = C.cast(self._res_b, C.POINTER(C.c_void_p))
            if getattr(cfg, "medusa_own_lm", False):
                self._medusa_lm = _ptr_array([weights[f"medusa.{i}.lm"] for i in range(cfg.n_medusa_heads)])
                w.medusa_lm = C.cast(self._medusa_lm, C.POINTER(C.c_void_p))
            if static_tree is None:
                raise ValueError("Medusa-style heads need a static tree (parent, level, rank)")
            self._st = [_i32_array(a) for a in static_tree]
            w.static_parent, w.static_level, w.static_rank = (C.cast(a, C.POINTER(C.c_int32)) for a in self._st)
        st = koala_state(self.target_k.data_ptr(), self.target_v.data_ptr(),
                         self.draft_k.data_ptr() if eagle and cfg.K > 0 else None,
                         self.draft_v.data_ptr() if eagle and cfg.K > 0 else None,
                         self.seq_len.data_ptr(), self.workspace.data_ptr() + self._ws_off, nbytes)
        self.stream = torch.cuda.current_stream(self.dev)
        rc = self.lib.koala_init(C.byref(self._cfg_c), C.byref(w), C.byref(st), self.stream.cuda_stream,
                                 C.byref(self._ctx))
        if rc != KOALA_OK:
            text = self.lib.koala_last_error(self._ctx).decode() if self._ctx else "koala_init"
            self.lib.koala_destroy(self._ctx)
            self._ctx = C.c_void_p(None)
            raise KoalaError(rc, text)
        self.out_stride = max(cfg.N, cfg.D + 1)
        self.out_tokens = torch.zeros(cfg.B, self.out_stride, dtype=torch.int32, device=self.dev)
        self.out_len = torch.zeros(cfg.B, dtype=torch.int32, device=self.dev)
        self._keep = None

    # ------------------------------------------------------------------ the five calls
    def _check(self, rc: int):
        if rc != KOALA_OK:
            raise KoalaError(rc, self.lib.koala_last_error(self._ctx).decode())

    def koala_draft(self, p: int):
        self._check(self.lib.koala_draft(self._ctx, p))

    def koala_expand_tree(self, p: int):
        self._check(self.lib.koala_expand_tree(self._ctx, p))

    def koala_verify(self, tree=None):
        """tree: None, or (tok [B, stride] int32 cuda, parent [B, stride] int32 cuda, n_nodes [B] int32 cuda, n_max)."""
        if tree is None:
            self._check(self.lib.koala_verify(self._ctx, None))
            return
        tok, parent, n_nodes, n_max = tree
        t = koala_tree(tok.data_ptr(), parent.data_ptr(), n_nodes.data_ptr(), tok.shape[1], int(n_max))
        self._keep = (tok, parent, n_nodes)
        self._check(self.lib.koala_verify(self._ctx, C.byref(t)))

    def koala_set_sampling(self, u_draft: Optional[torch.Tensor]):
        """u_draft: float32 device tensor [B][D] of uniforms (kept alive by the caller), or None."""
        self._u_draft = u_draft
        self._check(self.lib.koala_set_sampling(self._ctx, u_draft.data_ptr() if u_draft is not None else None))

    def koala_accept_sampled(self, u_accept: torch.Tensor, u_bonus: torch.Tensor):
        self._check(self.lib.koala_accept_sampled(self._ctx, u_accept.data_ptr(), u_bonus.data_ptr(),
                                                  self.out_tokens.data_ptr(), self.out_stride,
                                                  self.out_len.data_ptr()))
        return self.out_tokens, self.out_len

    def koala_accept_stats(self, n_max: int = 8, reset: bool = False):
        """(hits, trials) of the position-wise acceptance counters as two lists of n_max integers."""
        hits, trials = (C.c_uint64 * n_max)(), (C.c_uint64 * n_max)()
        self._check(self.lib.koala_accept_stats(self._ctx, hits, trials, n_max, 1 if reset else 0))
        return list(hits), list(trials)

    def koala_accept(self, forced_len: Optional[torch.Tensor] = None):
        """Returns (out_tokens [B, stride], out_len [B]) device tensors (asynchronous)."""
        self._check(self.lib.koala_accept(self._ctx, forced_len.data_ptr() if forced_len is not None else None,
                                          self.out_tokens.data_ptr(), self.out_stride, self.out_len.data_ptr()))
        self._keep_forced = forced_len
        return self.out_tokens, self.out_len

    def set_expand_mode(self, mode: int):
        self._check(self.lib.koala_set_option(self._ctx, 1, mode))

    def set_timing(self, on: bool):
        self._check(self.lib.koala_set_option(self._ctx, 2, int(on)))

    def timing(self) -> Dict[str, Dict[str, float]]:
        """Per kernel class: summed milliseconds, algorithmic bytes, launches (synchronises)."""
        t = koala_timing()
        self._check(self.lib.koala_timing_read(self._ctx, C.byref(t)))
        names = ("gemm_tc", "gemm_simt", "attention")
        return {n: {"ms": float(t.ms[i]), "bytes": int(t.bytes[i]), "launches": int(t.launches[i])}
                for i, n in enumerate(names)}

    def launch_count(self) -> int:
        return int(self.lib.koala_launch_count())

    def selftest_timeout(self, limit_cycles: int):
        """Diagnostic: enqueues a one-thread kernel whose bounded wait runs out (see koala_debug.h)."""
        self._check(self.lib.koala_selftest_timeout(self._ctx, int(limit_cycles)))

    def check_guards(self):
        """Diagnostic: (guards, damaged guards) of the workspace (synchronises the stream)."""
        n, bad = C.c_int(0), C.c_int(0)
        self._check(self.lib.koala_debug_check_guards(self._ctx, C.byref(n), C.byref(bad)))
        return n.value, bad.value

    def poll(self):
        done, status = C.c_int(0), C.c_int(0)
        self._check(self.lib.koala_poll(self._ctx, C.byref(done), C.byref(status)))
        return bool(done.value), status.value

    def device_status(self) -> int:
        """Synchronises the stream and returns the device status word."""
        self.stream.synchronize()
        self.poll()
        self.stream.synchronize()
        return self.poll()[1]

    # ------------------------------------------------------------------ workspace views
    def _view(self, ptr: int, shape, dtype) -> torch.Tensor:
        off = ptr - self.workspace.data_ptr()
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        return self.workspace[off:off + n].view(dtype).view(*shape)

    def buffers(self) -> Dict[str, torch.Tensor]:
        t = koala_buffer_table()
        self._check(self.lib.koala_buffers(self._ctx, C.byref(t)))
        c = self.cfg
        B, N, k, H, V, pool = c.B, c.N, c.topk, c.H, c.V, t.pool
        rows = max(t.draft_rows, 1)
        f32, i32 = torch.float32, torch.int32
        feat_shape = (c.n_medusa_heads * B, H) if c.head_kind == KOALA_MEDUSA else (B * k, H)
        spec = {"draft_logits": ((rows, V), f32), "draft_feat": (feat_shape, f32),
                "topk_tok": ((rows, k), i32), "topk_logp": ((rows, k), f32),
                "cand_tok": ((B, pool), i32), "cand_parent": ((B, pool), i32), "cand_score": ((B, pool), f32),
                "frontier": ((B, k), i32), "tree_tok": ((B, N), i32), "tree_parent": ((B, N), i32),
                "tree_level": ((B, N), i32), "tree_score": ((B, N), f32), "tree_n": ((B,), i32),
                "verify_logits": ((B * N, V), f32), "verify_hid": ((B * N, H), f32),
                "verify_tgt": ((B * N,), i32), "root_tok": ((B,), i32), "pend_hid": ((B, N, H), f32),
                "pend_tok": ((B, N), i32), "n_pend": ((B,), i32), "acc_path": ((B, N), i32)}
        return {name: self._view(getattr(t, name), shape, dt) for name, (shape, dt) in spec.items()}

    # ------------------------------------------------------------------ drivers (call sequencing only)
    def chain_tree(self, chunks: Sequence[Sequence[int]]):
        """Device arrays of one chain per sequence."""
        c = self.cfg
        n_max = max(len(x) for x in chunks)
        tok = np.zeros((c.B, n_max), np.int32)
        par = np.zeros((c.B, n_max), np.int32)
        for b, x in enumerate(chunks):
            tok[b, :len(x)] = x
            par[b, :len(x)] = np.arange(-1, len(x) - 1)
        n = np.asarray([len(x) for x in chunks], np.int32)
        to = lambda a: torch.from_numpy(a).to(self.dev)
        return to(tok), to(par), to(n), n_max

    def prefill(self, prompts: Sequence[Sequence[int]], chunk: int):
        """Ingests the prompts as chain trees with full forced acceptance (EAGLE-style heads also
        run draft pass 0 over every chunk but the last, with the next prompt token as root)."""
        c = self.cfg
        chunk = min(chunk, c.N)
        n_chunks = max(-(-len(p) // chunk) for p in prompts)
        parts = [np.array_split(np.asarray(p, dtype=np.int64), n_chunks) for p in prompts]
        bufs = self.buffers()
        for ci in range(n_chunks):
            tree = self.chain_tree([parts[b][ci] for b in range(c.B)])
            self.koala_verify(tree)
            self.koala_accept(tree[2])
            if c.head_kind == KOALA_EAGLE and ci + 1 < n_chunks:
                nxt = torch.tensor([int(parts[b][ci + 1][0]) for b in range(c.B)], dtype=torch.int32)
                bufs["root_tok"].copy_(nxt.to(self.dev))
                self.koala_draft(0)

    def step(self, forced_len: Optional[torch.Tensor] = None):
        """One whole iteration: D x (draft, expand_tree), verify, accept."""
        c = self.cfg
        passes = c.D if c.head_kind == KOALA_EAGLE else 1
        for p in range(passes):
            self.koala_draft(p)
            self.koala_expand_tree(p)
        self.koala_verify(None)
        return self.koala_accept(forced_len)

    def close(self):
        if self._ctx:
            torch.cuda.synchronize(self.dev)
            self.lib.koala_destroy(self._ctx)
            self._ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
