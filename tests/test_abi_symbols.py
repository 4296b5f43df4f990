"""The C-ABI library loads without a GPU and exports every function that
include/ap_serving.h declares."""
import ctypes
import os
import re

from paper_2604_07144_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ap_serving.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ap_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("ap_kv_pool_create", "ap_kv_append", "ap_attention_iteration"):
        assert must in names


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_functions()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} declared in ap_serving.h but not exported"
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_status_strings():
    assert binding.status_string(0) == "ok"
    assert "block table" in binding.status_string(binding.AP_ERR_BAD_BLOCK_TABLE)
    assert binding.kv_pool_bytes(10, 8, 128) == 10 * 8 * 16 * 128 * 2
    assert binding.kv_pool_bytes(0, 8, 128) == 0
