"""The C-ABI library loads without a GPU and exports every entry point the header declares."""
import ctypes
import os
import re

import paper_2401_04836_b200 as cb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    with open(os.path.join(ROOT, "include", "const_b200.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(const_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"const_csf_build", "const_plan_create", "const_execute", "const_destroy"} <= set(names)
    lib = ctypes.CDLL(cb.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_binding_mirrors_the_header():
    for n in _declared():
        assert hasattr(cb, n), n


def test_status_strings_and_null_handling():
    lib = cb.load_library()
    seen = {cb.const_status_string(s) for s in range(9)}
    assert len(seen) == 9 and "ok" in seen
    lib.const_destroy(None)                                   # NULL is a no-op
    out = ctypes.c_void_p()
    assert lib.const_plan_create(None, None, 0, None, None, 0, None, None, 0, 0, ctypes.byref(out)) == 1
    assert lib.const_csf_build(3, None, 0, None, None, 0, None, None, ctypes.byref(out)) == 1
    assert lib.const_execute(None, None, 0, None, None) == 1
    assert lib.const_csf_level(None, 0, None, None, None) == 1
