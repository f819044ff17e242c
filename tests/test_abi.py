"""The C-ABI library builds for sm_100a, loads without a GPU and exports what include/*.h declares."""
import ctypes
import glob
import os
import re

from paper_2512_22560_b200 import build as rbuild
from paper_2512_22560_b200 import rollart

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = open(h).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(rollart_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = rbuild.build()
    lib = ctypes.CDLL(lib_path)
    decl = declared_symbols()
    assert {"rollart_kv_append", "rollart_decode_attn", "rollart_obs_chunk_attn", "rollart_create", "rollart_destroy",
            "rollart_workspace_size", "rollart_check", "rollart_last_error"} <= decl
    for name in decl:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert decl == set(rollart.EXPORTS) or decl >= set(rollart.EXPORTS)
    for name in rollart.EXPORTS:
        assert name in decl


def test_workspace_size_is_host_arithmetic():
    a = rollart.workspace_size(64, 28, 4, 16384)
    b = rollart.workspace_size(256, 64, 8, 32768)
    assert 0 < a < b < (1 << 32)
    assert rollart.workspace_size(0, 8, 2, 100) == 0


def test_null_context_is_rejected_without_a_gpu():
    lib = rollart.load_library()
    assert lib.rollart_check(None, None) == rollart.ERR_INVALID_ARG
    assert lib.rollart_destroy(None) == rollart.ERR_INVALID_ARG
    assert lib.rollart_last_error(None) == b"context is NULL"


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_22560_b200")
    for path in glob.glob(os.path.join(pkg, "**", "*"), recursive=True):
        if os.path.isfile(path) and path.endswith((".py", ".cu", ".cuh", ".h")):
            text = open(path).read()
            assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), path
            assert "rollart_oracle" not in text, path
