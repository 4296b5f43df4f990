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


def test_header_is_plain_c_and_struct_sizes_match_the_binding(tmp_path):
    """include/ap_serving.h compiles as C99 on its own, and the structs the ctypes binding mirrors have
    the sizes (and the enum the values) a C compiler gives them."""
    import subprocess
    src = tmp_path / "sizes.c"
    src.write_text(
        '#include "ap_serving.h"\n#include <stdio.h>\n'
        "int main(void) {\n"
        '  printf("%zu %zu %zu %zu %zu %zu %d %d %d\\n", sizeof(ap_pool_desc), sizeof(ap_batch_desc), sizeof(ap_plan_info),\n'
        "         sizeof(ap_plan_prediction), sizeof(ap_plan_layout), sizeof(ap_kernel_times), (int)AP_KERNEL_COUNT,\n"
        "         (int)AP_ERR_UNSUPPORTED, (int)AP_STATIC_WORKSPACE_BYTES);\n"
        "  return 0;\n}\n")
    exe = tmp_path / "sizes"
    inc = os.path.join(ROOT, "include")
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", inc, "-fsyntax-only", "-x", "c",
                           os.path.join(inc, "ap_serving.h")])
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", inc, str(src), "-o", str(exe)])
    got = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    want = [ctypes.sizeof(binding.PoolDesc), ctypes.sizeof(binding.BatchDesc), ctypes.sizeof(binding.PlanInfo),
            ctypes.sizeof(binding.PlanPrediction), ctypes.sizeof(binding.PlanLayout), ctypes.sizeof(binding.KernelTimes),
            len(binding.KERNEL_NAMES), binding.AP_ERR_UNSUPPORTED, 8 << 20]
    assert got == want
