"""The C-ABI library loads and exports every function its header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            text = open(os.path.join(ROOT, "include", f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(fp_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    from paper_2010_16165_b200 import build, binding
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"fp_fuse", "fp_prune", "fp_forward", "fp_forward_host", "fp_forward_host_async", "fp_score", "fp_query", "fp_destroy",
            "fp_last_error"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(binding.EXPORTS) <= names


def test_struct_layouts_match_header():
    from paper_2010_16165_b200 import binding
    assert ctypes.sizeof(binding.fp_node) == 80
    assert binding.fp_node.w_off.offset == 56
    assert ctypes.sizeof(binding.fp_op_info) == 16 * 4 + 3 * 8 + 2 * 4
    assert binding.fp_op_info.chain.offset == 16 * 4 + 3 * 8
    assert binding.fp_model_desc.nodes.offset == 8


def test_null_arguments_are_rejected_without_a_gpu():
    from paper_2010_16165_b200 import binding
    lib = binding.lib()
    assert lib.fp_fuse(None, None, 0, None, 0, 1, None) == binding.FP_ERR_ARG
    assert b"NULL" in lib.fp_last_error()
    assert lib.fp_forward(None, None, 1, None, None) == binding.FP_ERR_ARG
    assert lib.fp_destroy(None) == binding.FP_OK
