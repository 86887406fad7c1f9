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


def test_execute_refuses_misaligned_pointers_before_touching_the_device():
    """Dense operands and the output are read and written with 128-bit accesses: a pointer that is not
    16-byte aligned is refused with CONST_ERR_INVALID_ARG before any device call."""
    import torch
    from workloads import make_config
    w = make_config(1)
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    lib = ctypes.CDLL(cb.library_path())                      # its own function objects: the binding's prototypes stay as they are

    class Operand(ctypes.Structure):
        _fields_ = [("name", ctypes.c_char_p), ("csf", ctypes.c_void_p), ("dense_dev", ctypes.c_void_p)]

    fake_csf = ctypes.create_string_buffer(1024)              # zeroed: not a CSF handle (wrong magic)
    base = 0x7f0000001000                                     # never dereferenced on the paths below

    def run(u_ptr, v_ptr, out_ptr):
        ops = (Operand * 3)(Operand(b"X", ctypes.addressof(fake_csf), None), Operand(b"U", None, u_ptr),
                            Operand(b"V", None, v_ptr))
        return lib.const_execute(ctypes.c_void_p(plan.ptr), ctypes.cast(ops, ctypes.c_void_p), 3,
                                 ctypes.c_void_p(out_ptr), None)

    lib.const_execute.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    assert run(base + 4, base, base) == 1                     # factor row base off by one float
    assert run(base, base + 8, base) == 1
    assert run(base, base, base + 4) == 1                     # output
    aligned = run(base, base, base)
    if not torch.cuda.is_available():
        assert aligned == 7                                   # got past the alignment check to the first device call
    else:
        assert aligned == 1                                   # the fake CSF handle is refused; nothing was launched
