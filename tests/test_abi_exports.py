"""The C-ABI library builds, loads without a GPU and exports every symbol include/moe_pd.h declares."""
import ctypes
import os
import re

from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moe_pd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    build_mod.build_library()
    lib = B.load_library()
    declared = _declared()
    assert declared == sorted(B.EXPORTS), "binding.EXPORTS and the header disagree"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"
    assert "sm_100a" in B.moe_version()


def test_host_only_entry_points_work_without_a_gpu():
    cfg = B.make_config(7168, 256, 8, 2048, 2048, 128, B.MOE_PHASE_DECODE)
    n = B.moe_ctx_workspace_bytes(cfg)
    cfg_p = B.make_config(7168, 256, 8, 2048, 2048, 128, B.MOE_PHASE_PREFILL)
    n_p = B.moe_ctx_workspace_bytes(cfg_p)
    # x_perm + y_perm alone are 2 * N * H * 2 bytes; a D context holds two buffer sets, a P context one; both add
    # staging slots for the pipelined host path (logits, x and out of one batch each) up to four in all
    staging = 128 * 256 * 4 + 2 * 128 * 7168 * 2
    assert n_p >= 2 * 128 * 8 * 7168 * 2 and n - 2 * staging > 1.9 * (n_p - 3 * staging) - 4096
    assert B.moe_ctx_workspace_bytes(B.make_config(100, 8, 2, 128, 0, 4)) == 0
    lib = B.load_library()
    bad = B.make_config(256, 8, 9, 128, 0, 4)  # k > E: refused before any CUDA call
    h = ctypes.c_void_p()
    assert lib.moe_ctx_create(ctypes.byref(bad), None, 0, None, ctypes.byref(h)) == B.MOE_ERR_INVALID_ARG
    assert b"top_k" in lib.moe_last_error(None)
    assert lib.moe_ctx_destroy(None) == B.MOE_ERR_INVALID_ARG
    assert lib.moe_route(None, None, None, 0, None, None) == B.MOE_ERR_INVALID_ARG


def test_no_product_code_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_00993_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), f
                assert "moe_oracle" not in text, f
