"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2609_21137_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(moe_vqlr_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_builds_and_exports_declared_symbols():
    path = build.build_library()
    lib = ctypes.CDLL(path)
    declared = _declared_symbols()
    assert {"moe_vqlr_create", "moe_vqlr_decode_layer", "moe_vqlr_destroy"} <= declared
    for name in declared:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2609_21137_b200 import binding
    assert set(binding.EXPORTS) == _declared_symbols()


def test_create_rejects_bad_arguments_without_a_gpu():
    from paper_2609_21137_b200 import binding
    lib = binding.library()
    h = ctypes.c_void_p()
    assert lib.moe_vqlr_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    cfg = binding._Config()
    assert lib.moe_vqlr_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert h.value is None
    assert lib.moe_vqlr_last_error(None)
    assert lib.moe_vqlr_destroy(None) == binding.OK
    assert lib.moe_vqlr_decode_layer(None, None, 1, None, None, None) == binding.ERR_INVALID_ARG
