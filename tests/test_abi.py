"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes as C
import os
import re

from paper_2408_08146_b200 import binding
from workloads import CONFIGS, TINY_EAGLE, TINY_MEDUSA

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "koala.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(koala_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    names = _declared_symbols()
    assert {"koala_init", "koala_draft", "koala_expand_tree", "koala_verify", "koala_accept"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"libkoala.so does not export {n}"


def test_struct_layouts_match_the_header_sizes():
    # 4-byte fields only in koala_config; pointer tables elsewhere
    assert C.sizeof(binding.koala_config) == 19 * 4
    assert C.sizeof(binding.koala_tree) == 3 * 8 + 2 * 4
    assert C.sizeof(binding.koala_buffer_table) == 21 * 8 + 2 * 4


def test_workspace_size_and_config_validation():
    for cfg in CONFIGS + [TINY_MEDUSA]:
        assert binding.koala_workspace_bytes(cfg) > 0, cfg.name
    assert binding.koala_workspace_bytes(TINY_EAGLE.with_(head_dim=48, n_heads=4, H=192)) == 0
    assert binding.koala_workspace_bytes(TINY_EAGLE.with_(N=129)) == 0
    assert binding.koala_workspace_bytes(TINY_EAGLE.with_(topk=17)) == 0
    assert binding.koala_workspace_bytes(TINY_MEDUSA.with_(D=2)) == 0          # D != heads
    assert binding.koala_workspace_bytes(TINY_EAGLE.with_(D=10, topk=16)) == 0  # (D-1)*k > 128
    # bigger trees and batches need more workspace
    assert binding.koala_workspace_bytes(TINY_EAGLE.with_(B=2)) > binding.koala_workspace_bytes(TINY_EAGLE)


def test_init_rejects_bad_arguments_before_touching_the_device():
    lib = binding.load_library()
    ctx = C.c_void_p(None)
    cfg = binding.make_config(TINY_EAGLE.with_(N=0))
    w, st = binding.koala_weights(), binding.koala_state()
    rc = lib.koala_init(C.byref(cfg), C.byref(w), C.byref(st), None, C.byref(ctx))
    assert rc == 1 and b"N out of range" in lib.koala_last_error(ctx)
    lib.koala_destroy(ctx)
    cfg = binding.make_config(TINY_EAGLE)
    rc = lib.koala_init(C.byref(cfg), C.byref(w), C.byref(st), None, C.byref(ctx))
    assert rc == 1 and b"missing target weights" in lib.koala_last_error(ctx)
    lib.koala_destroy(ctx)
    assert lib.koala_draft(None, 0) == 1 and lib.koala_verify(None, None) == 1
    assert lib.koala_gemm_bf16(None, None, None, None, 0, 0, 0, 0, None, 0, 1, 0, None, None) == 1
