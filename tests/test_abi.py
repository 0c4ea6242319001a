"""CPU-side checks of the boundary: the library builds/loads and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            src = open(os.path.join(ROOT, "include", f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(moa_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    names = declared_functions()
    assert {"moa_lsa_forward", "moa_draft_step", "moa_tree_expand", "moa_tree_attn_mask"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(moa.EXPORTS) == sorted(n for n in names)


def test_status_strings_and_struct_sizes():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    assert lib.moa_status_str(0) == b"ok"
    assert lib.moa_status_str(5) == b"workspace too small"
    assert ctypes.sizeof(moa.MoaConfig) == 22 * 4
    assert ctypes.sizeof(moa.MoaWeights) == 31 * 8
    assert ctypes.sizeof(moa.MoaState) == 9 * 8 + 8   # nine pointers, int32 + padding


def test_null_arguments_are_rejected_without_a_gpu():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    assert lib.moa_create(None, None, None) == 1
    assert lib.moa_tree_attn_mask(None, 1, 4, None, 0, None) == 1
    assert lib.moa_state_bytes(None, 1, None, None) == 1
    lib.moa_destroy(None)


def test_product_path_has_no_oracle_or_cpu_fallback():
    pkg = os.path.join(ROOT, "paper_2410_03804_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "synth.py", f
