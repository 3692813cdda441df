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


def test_debug_header_symbols_are_exported_too():
    """The diagnostic exports (tuning, launch counter, timeout self-test, workspace guards) are
    declared outside the interface, in csrc/koala_debug.h, and exported by the same library."""
    text = open(os.path.join(ROOT, "paper_2408_08146_b200", "csrc", "koala_debug.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = sorted(set(re.findall(r"\b(koala_[a-z0-9_]+)\s*\(", text)))
    assert {"koala_set_tuning", "koala_launch_count", "koala_selftest_timeout", "koala_debug_check_guards"} <= set(names)
    lib = binding.load_library()
    for n in names:
        assert hasattr(lib, n), f"libkoala.so does not export {n}"
    # none of them is declared in the interface header
    assert not set(names) & set(_declared_symbols())


def test_token_tile_rows_of_the_standalone_multiply():
    """koala_gemm_x_rows: whole token tiles - multiples of 16 up to 128 tokens; beyond that 256-token
    tiles for plain operands and for pairs (which keep value and residual in one accumulator there)."""
    lib = binding.load_library()
    rows = lambda m, pair: int(lib.koala_gemm_x_rows(m, pair))
    assert [rows(m, 1) for m in (1, 16, 17, 64, 100, 128)] == [16, 16, 32, 64, 112, 128]
    assert [rows(m, 1) for m in (129, 200, 256, 257, 512)] == [144, 208, 256, 512, 512]
    assert [rows(m, 0) for m in (10, 128, 129, 256, 300)] == [16, 128, 144, 256, 512]
    assert rows(0, 1) == 0
    assert int(lib.koala_gemm_static_scratch_bytes()) == 8 << 20
