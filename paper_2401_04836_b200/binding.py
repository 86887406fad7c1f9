"""ctypes binding of the C ABI declared in include/const_b200.h.

Function names mirror the C entry points.  Tensors are torch CUDA tensors (torch supplies device
memory and streams only); the binding passes their data pointers through.  There is no CPU
fallback: if the shared library is missing the import of this module's functions fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence, Tuple, Union

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libconst_b200.so"

F32, F64 = 0, 1
STATUS_NAMES = {0: "CONST_OK", 1: "CONST_ERR_INVALID_ARG", 2: "CONST_ERR_UNSUPPORTED",
                3: "CONST_ERR_ILLEGAL_SCHEDULE", 4: "CONST_ERR_DUPLICATE_COORD", 5: "CONST_ERR_COORD_RANGE",
                6: "CONST_ERR_WORKSPACE", 7: "CONST_ERR_CUDA", 8: "CONST_ERR_TIMEOUT"}


class ConstError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {STATUS_NAMES.get(self.status, self.status)} "
                         f"({const_status_string(self.status)})")


class _Extent(ctypes.Structure):
    _fields_ = [("index", ctypes.c_char), ("extent", ctypes.c_int64)]


class _Operand(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char_p), ("csf", ctypes.c_void_p), ("dense_dev", ctypes.c_void_p)]


_lib = None


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Load libconst_b200.so (built in-tree by paper_2401_04836_b200/build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2401_04836_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    pp = ctypes.POINTER
    lib.const_csf_build.argtypes = [i32, pp(i64), i64, pp(vp), vp, i32, pp(i32), vp, pp(vp)]
    lib.const_csf_from_dense.argtypes = [i32, pp(i64), vp, i32, pp(i32), vp, pp(vp)]
    lib.const_csf_from_dense.restype = i32
    lib.const_csf_build_noalloc.argtypes = [i32, pp(i64), i64, pp(vp), vp, i32, pp(i32), vp, pp(vp), pp(vp), vp,
                                            pp(i64)]
    lib.const_csf_build_noalloc.restype = i32
    lib.const_csf_level.argtypes = [vp, i32, pp(vp), pp(vp), pp(i64)]
    lib.const_csf_values.argtypes = [vp, pp(vp), pp(i64)]
    lib.const_csf_set_bins.argtypes = [vp, i64, i64, i64, vp]
    lib.const_csf_bin_counts.argtypes = [vp, pp(i64), pp(i64), pp(i64), pp(i64)]
    lib.const_csf_work_lists.argtypes = [vp, pp(vp), pp(vp), pp(i64), pp(vp), pp(i64)]
    lib.const_csf_work_lists.restype = i32
    lib.const_microbench.argtypes = [i32, vp, i64, i64, i32, i32, vp, pp(ctypes.c_double), pp(ctypes.c_double)]
    lib.const_microbench.restype = i32
    lib.const_debug_set.argtypes = [i32, i64]
    lib.const_debug_set.restype = i32
    lib.const_plan_create.argtypes = [ctypes.c_char_p, pp(ctypes.c_char_p), i32, pp(ctypes.c_char_p),
                                      pp(pp(i32)), i32, pp(ctypes.c_char_p), pp(_Extent), i32, i32, pp(vp)]
    lib.const_schedule_check.argtypes = [ctypes.c_char_p, pp(ctypes.c_char_p), i32, pp(ctypes.c_char_p),
                                         pp(pp(i32)), i32, pp(ctypes.c_char_p), pp(_Extent), i32, pp(i32)]
    lib.const_schedule_cin.argtypes = [ctypes.c_char_p, pp(ctypes.c_char_p), i32, pp(ctypes.c_char_p),
                                       pp(pp(i32)), i32, pp(ctypes.c_char_p), pp(_Extent), i32, i32, ctypes.c_char_p,
                                       i64, pp(i64)]
    lib.const_schedule_cin.restype = i32
    lib.const_plan_reduced_order.argtypes = [vp, i32, pp(i32)]
    lib.const_plan_family.argtypes = [vp]
    lib.const_plan_family.restype = ctypes.c_char_p
    lib.const_execute.argtypes = [vp, pp(_Operand), i32, vp, vp]
    lib.const_last_device_status.argtypes = [vp, vp]
    lib.const_plan_set_tensor_stage.argtypes = [vp, i32]
    lib.const_plan_set_tensor_stage.restype = i32
    lib.const_plan_describe.argtypes = [vp, ctypes.c_char_p, i64, pp(i64)]
    lib.const_plan_describe.restype = i32
    lib.const_plan_set_generic_executor.argtypes = [vp, i32]
    lib.const_plan_set_generic_executor.restype = i32
    lib.const_destroy.argtypes = [vp]
    lib.const_destroy.restype = None
    lib.const_profile_enable.argtypes = [i32]
    lib.const_profile_enable.restype = i32
    lib.const_profile_read.argtypes = [ctypes.c_char_p, i64, pp(i64), pp(ctypes.c_double), i32, pp(i32)]
    lib.const_profile_read.restype = i32
    lib.const_status_string.argtypes = [i32]
    lib.const_status_string.restype = ctypes.c_char_p
    for name in ("const_csf_build", "const_csf_level", "const_csf_values", "const_csf_set_bins",
                 "const_csf_bin_counts", "const_plan_create", "const_schedule_check", "const_plan_reduced_order", "const_execute",
                 "const_last_device_status"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def const_status_string(status: int) -> str:
    return load_library().const_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise ConstError(status, where)


def _stream_ptr(stream) -> ctypes.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(int(getattr(stream, "cuda_stream", stream)))


class CsfHandle:
    """Owns a const_csf_t*; `order`, `dtype` mirror the build arguments."""

    def __init__(self, ptr: int, order: int, dtype: int):
        self.ptr, self.order, self.dtype = ptr, order, dtype

    def __del__(self):
        try:
            const_destroy(self)
        except Exception:
            pass


class PlanHandle:
    def __init__(self, ptr: int):
        self.ptr = ptr

    def __del__(self):
        try:
            const_destroy(self)
        except Exception:
            pass


def const_csf_build(coords, vals, dims: Sequence[int], mode_order: Sequence[int], stream=None) -> CsfHandle:
    """coords: one int32 CUDA tensor per mode; vals: float32/float64 CUDA tensor."""
    import torch
    lib = load_library()
    order = len(dims)
    if len(coords) != order or len(mode_order) != order:
        raise ValueError("coords, dims and mode_order must have one entry per mode")
    nnz = int(vals.numel())
    for c in coords:
        if c.dtype != torch.int32 or not c.is_cuda or not c.is_contiguous() or c.numel() != nnz:
            raise ValueError("coordinates must be contiguous int32 CUDA tensors of nnz entries")
    if not vals.is_cuda or not vals.is_contiguous() or vals.dtype not in (torch.float32, torch.float64):
        raise ValueError("values must be a contiguous float32/float64 CUDA tensor")
    dtype = F32 if vals.dtype == torch.float32 else F64
    dims_a = (ctypes.c_int64 * order)(*[int(d) for d in dims])
    mo_a = (ctypes.c_int * order)(*[int(m) for m in mode_order])
    cptr = (ctypes.c_void_p * order)(*[c.data_ptr() for c in coords])
    out = ctypes.c_void_p()
    st = lib.const_csf_build(order, dims_a, nnz, cptr, ctypes.c_void_p(vals.data_ptr()), dtype, mo_a,
                             _stream_ptr(stream), ctypes.byref(out))
    _check(st, "const_csf_build")
    return CsfHandle(out.value, order, dtype)


def const_csf_from_dense(dense, mode_order: Sequence[int], stream=None) -> CsfHandle:
    """dense: contiguous float32/float64 CUDA tensor; its entries that are not zero become the CSF tensor's nonzeros."""
    import torch
    lib = load_library()
    if not dense.is_cuda or not dense.is_contiguous() or dense.dtype not in (torch.float32, torch.float64):
        raise ValueError("dense must be a contiguous float32/float64 CUDA tensor")
    order = dense.dim()
    dtype = F32 if dense.dtype == torch.float32 else F64
    dims_a = (ctypes.c_int64 * order)(*[int(d) for d in dense.shape])
    mo_a = (ctypes.c_int * order)(*[int(m) for m in mode_order])
    out = ctypes.c_void_p()
    _check(lib.const_csf_from_dense(order, dims_a, ctypes.c_void_p(dense.data_ptr()), dtype, mo_a, _stream_ptr(stream),
                                    ctypes.byref(out)), "const_csf_from_dense")
    return CsfHandle(out.value, order, dtype)


def const_csf_build_noalloc(coords, vals, dims: Sequence[int], mode_order: Sequence[int], pos_out, crd_out,
                            vals_out, stream=None) -> List[int]:
    """COO -> CSF into buffers the caller owns, for callers that may not allocate device memory.

    pos_out / crd_out: one int32 CUDA tensor per level with room for nnz + 1 / nnz entries;
    vals_out: CUDA tensor like `vals`.  Nothing is allocated on the device by this call (the
    library's temporaries sit in a fixed static array, which limits nnz to 262 144).
    Returns the number of nodes per level.
    """
    import torch
    lib = load_library()
    order = len(dims)
    nnz = int(vals.numel())
    dtype = F32 if vals.dtype == torch.float32 else F64
    for l in range(order):
        if pos_out[l].dtype != torch.int32 or crd_out[l].dtype != torch.int32:
            raise ValueError("pos/crd outputs must be int32")
        if pos_out[l].numel() < (2 if l == 0 else nnz + 1) or crd_out[l].numel() < nnz:
            raise ValueError("output buffer too small")
    if vals_out.dtype != vals.dtype or vals_out.numel() < nnz:
        raise ValueError("vals_out must match vals")
    dims_a = (ctypes.c_int64 * order)(*[int(d) for d in dims])
    mo_a = (ctypes.c_int * order)(*[int(m) for m in mode_order])
    cptr = (ctypes.c_void_p * order)(*[c.data_ptr() for c in coords])
    pptr = (ctypes.c_void_p * order)(*[p.data_ptr() for p in pos_out])
    rptr = (ctypes.c_void_p * order)(*[c.data_ptr() for c in crd_out])
    sizes = (ctypes.c_int64 * order)()
    st = lib.const_csf_build_noalloc(order, dims_a, nnz, cptr, ctypes.c_void_p(vals.data_ptr()), dtype, mo_a,
                                     _stream_ptr(stream), pptr, rptr, ctypes.c_void_p(vals_out.data_ptr()), sizes)
    _check(st, "const_csf_build_noalloc")
    return list(sizes)


def _dev_to_torch(ptr: Optional[int], n: int, dtype):
    """Copy n elements from a borrowed device pointer into a fresh torch CUDA tensor."""
    import torch
    out = torch.empty(n, dtype=dtype, device="cuda")
    if n:
        cudart = ctypes.CDLL("libcudart.so.12")
        cudart.cudaMemcpy.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
        torch.cuda.synchronize()
        rc = cudart.cudaMemcpy(out.data_ptr(), ptr, n * out.element_size(), 3)   # cudaMemcpyDeviceToDevice
        if rc != 0:
            raise RuntimeError(f"cudaMemcpy failed with {rc}")
    return out


def const_csf_level(csf: CsfHandle, level: int):
    """Returns (pos, crd) of one level as torch int32 CUDA tensors (copies of the library's arrays)."""
    import torch
    lib = load_library()
    pos, crd, n = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_int64()
    _check(lib.const_csf_level(csf.ptr, level, ctypes.byref(pos), ctypes.byref(crd), ctypes.byref(n)),
           "const_csf_level")
    if level == 0:
        n_pos = 2
    else:
        prev = ctypes.c_int64()
        _check(lib.const_csf_level(csf.ptr, level - 1, None, None, ctypes.byref(prev)), "const_csf_level")
        n_pos = prev.value + 1
    return _dev_to_torch(pos.value, n_pos, torch.int32), _dev_to_torch(crd.value, n.value, torch.int32)


def const_csf_values(csf: CsfHandle):
    import torch
    lib = load_library()
    vals, nnz = ctypes.c_void_p(), ctypes.c_int64()
    _check(lib.const_csf_values(csf.ptr, ctypes.byref(vals), ctypes.byref(nnz)), "const_csf_values")
    return _dev_to_torch(vals.value, nnz.value, torch.float32 if csf.dtype == F32 else torch.float64)


def const_csf_set_bins(csf: CsfHandle, light_max_nnz: int = 0, heavy_max_nnz: int = 0, chunk_nnz: int = 0,
                       stream=None) -> None:
    _check(load_library().const_csf_set_bins(csf.ptr, int(light_max_nnz), int(heavy_max_nnz), int(chunk_nnz),
                                             _stream_ptr(stream)), "const_csf_set_bins")


def const_csf_bin_counts(csf: CsfHandle) -> Dict[str, int]:
    a, b, c, d = (ctypes.c_int64() for _ in range(4))
    _check(load_library().const_csf_bin_counts(csf.ptr, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                               ctypes.byref(d)), "const_csf_bin_counts")
    return {"light": a.value, "heavy": b.value, "giant": c.value, "items": d.value}


def const_csf_work_lists(csf: CsfHandle):
    """Copies of the load balancer's lists: (slice_ptr [n0+1], light_list [n_light], items [n_items, 4]) as int32 CUDA tensors."""
    import torch
    lib = load_library()
    sp, ll, it = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
    n_light, n_items, n0 = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(lib.const_csf_work_lists(csf.ptr, ctypes.byref(sp), ctypes.byref(ll), ctypes.byref(n_light), ctypes.byref(it),
                                    ctypes.byref(n_items)), "const_csf_work_lists")
    _check(lib.const_csf_level(csf.ptr, 0, None, None, ctypes.byref(n0)), "const_csf_level")
    return (_dev_to_torch(sp.value, n0.value + 1 if n0.value else 0, torch.int32),
            _dev_to_torch(ll.value, n_light.value, torch.int32),
            _dev_to_torch(it.value, 4 * n_items.value, torch.int32).reshape(-1, 4))


BENCH_FP32_FMA, BENCH_FP64_FMA, BENCH_TF32_MMA, BENCH_ROW_GATHER, BENCH_FP64_MMA = 0, 1, 2, 3, 4


def const_microbench(kind: int, rows=None, table_rows: int = 0, rank: int = 0, repeats: int = 5, stream=None):
    """Machine-limit micro-benchmark (see the header); returns (milliseconds per launch, work per launch)."""
    ms, work = ctypes.c_double(), ctypes.c_double()
    ptr, n = (None, 0) if rows is None else (ctypes.c_void_p(rows.data_ptr()), int(rows.numel()))
    _check(load_library().const_microbench(int(kind), ptr, n, int(table_rows), int(rank), int(repeats),
                                           _stream_ptr(stream), ctypes.byref(ms), ctypes.byref(work)), "const_microbench")
    return ms.value, work.value


def const_debug_set(what: int, value: int) -> None:
    """Test hook: limits of the bounded device-side waits (see the header)."""
    _check(load_library().const_debug_set(int(what), int(value)), "const_debug_set")


def _schedule_args(tree, mode_orders, loop_orders, extents):
    n_c = len(tree)
    if len(loop_orders) != n_c:
        raise ValueError("one loop order per contraction")
    tree_a = (ctypes.c_char_p * n_c)(*[t.encode() for t in tree])
    loops_a = (ctypes.c_char_p * n_c)(*[s.encode() for s in loop_orders])
    names = list(mode_orders)
    names_a = (ctypes.c_char_p * max(len(names), 1))(*[n.encode() for n in names])
    mo_arrays = [(ctypes.c_int * len(mode_orders[n]))(*[int(x) for x in mode_orders[n]]) for n in names]
    mo_a = (ctypes.POINTER(ctypes.c_int) * max(len(names), 1))(
        *[ctypes.cast(a, ctypes.POINTER(ctypes.c_int)) for a in mo_arrays])
    ext_a = (_Extent * len(extents))(*[_Extent(k.encode(), int(v)) for k, v in extents.items()])
    return tree_a, n_c, names_a, mo_a, len(names), loops_a, ext_a, len(extents), mo_arrays


def const_schedule_check(expression: str, tree: Sequence[str], mode_orders: Dict[str, Sequence[int]],
                         loop_orders: Sequence[str], extents: Dict[str, int]) -> List[int]:
    """Host-only legality check (Sec. 3.2); returns the reduced order of every contraction's result."""
    lib = load_library()
    tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e, _keep = _schedule_args(tree, mode_orders, loop_orders, extents)
    red = (ctypes.c_int * n_c)()
    _check(lib.const_schedule_check(expression.encode(), tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e, red),
           "const_schedule_check")
    return list(red)


def const_schedule_cin(expression: str, tree: Sequence[str], mode_orders: Dict[str, Sequence[int]],
                       loop_orders: Sequence[str], extents: Dict[str, int], validate: bool = True) -> str:
    """Host-only: concrete index notation (forall / where nest) of the schedule, Algorithm 1 of Sec. 4.2."""
    lib = load_library()
    tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e, _keep = _schedule_args(tree, mode_orders, loop_orders, extents)
    need = ctypes.c_int64()
    args = (expression.encode(), tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e, 1 if validate else 0)
    _check(lib.const_schedule_cin(*args, None, 0, ctypes.byref(need)), "const_schedule_cin")
    buf = ctypes.create_string_buffer(max(int(need.value), 1))
    _check(lib.const_schedule_cin(*args, buf, len(buf), ctypes.byref(need)), "const_schedule_cin")
    return buf.value.decode()


def const_plan_create(expression: str, tree: Sequence[str], mode_orders: Dict[str, Sequence[int]],
                      loop_orders: Sequence[str], extents: Dict[str, int], dtype: int) -> PlanHandle:
    """Host-only: parses and checks the schedule, binds a kernel family.  Needs no GPU."""
    lib = load_library()
    tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e, _keep = _schedule_args(tree, mode_orders, loop_orders, extents)
    out = ctypes.c_void_p()
    st = lib.const_plan_create(expression.encode(), tree_a, n_c, names_a, mo_a, n_s, loops_a, ext_a, n_e,
                               int(dtype), ctypes.byref(out))
    _check(st, "const_plan_create")
    return PlanHandle(out.value)


def const_plan_reduced_order(plan: PlanHandle, contraction: int) -> int:
    o = ctypes.c_int()
    _check(load_library().const_plan_reduced_order(plan.ptr, contraction, ctypes.byref(o)), "const_plan_reduced_order")
    return o.value


def const_plan_family(plan: PlanHandle) -> str:
    return load_library().const_plan_family(plan.ptr).decode()


def const_execute(plan: PlanHandle, operands: Dict[str, Union[CsfHandle, "object"]], out, stream=None) -> None:
    """operands: name -> CsfHandle or dense torch CUDA tensor (row-major).  `out` is overwritten."""
    lib = load_library()
    ops = (_Operand * len(operands))()
    keep = []
    for slot, (name, val) in zip(ops, operands.items()):
        b = name.encode()
        keep.append(b)
        slot.name = b
        if isinstance(val, CsfHandle):
            slot.csf, slot.dense_dev = val.ptr, None
        else:
            if not val.is_cuda or not val.is_contiguous():
                raise ValueError(f"dense operand {name} must be a contiguous CUDA tensor")
            slot.csf, slot.dense_dev = None, val.data_ptr()
    if not out.is_cuda or not out.is_contiguous():
        raise ValueError("output must be a contiguous CUDA tensor")
    _check(lib.const_execute(plan.ptr, ops, len(operands), ctypes.c_void_p(out.data_ptr()), _stream_ptr(stream)),
           "const_execute")


def const_plan_set_tensor_stage(plan: PlanHandle, enable: bool) -> None:
    _check(load_library().const_plan_set_tensor_stage(plan.ptr, 1 if enable else 0), "const_plan_set_tensor_stage")


def const_plan_describe(plan: PlanHandle) -> str:
    """Listing of what the generic executor does for this plan (loops, drivers, workspaces)."""
    lib = load_library()
    need = ctypes.c_int64()
    _check(lib.const_plan_describe(plan.ptr, None, 0, ctypes.byref(need)), "const_plan_describe")
    buf = ctypes.create_string_buffer(max(int(need.value), 1))
    _check(lib.const_plan_describe(plan.ptr, buf, len(buf), ctypes.byref(need)), "const_plan_describe")
    return buf.value.decode()


def const_plan_set_generic_executor(plan: PlanHandle, enable: bool) -> None:
    _check(load_library().const_plan_set_generic_executor(plan.ptr, 1 if enable else 0), "const_plan_set_generic_executor")


def const_last_device_status(plan: PlanHandle, stream=None) -> int:
    return int(load_library().const_last_device_status(plan.ptr, _stream_ptr(stream)))


def const_destroy(handle) -> None:
    """Release a CsfHandle or PlanHandle (idempotent)."""
    if handle is None or getattr(handle, "ptr", None) is None:
        return
    ptr, handle.ptr = handle.ptr, None
    if _lib is not None:
        _lib.const_destroy(ctypes.c_void_p(ptr))


def const_profile_enable(on: bool) -> None:
    _check(load_library().const_profile_enable(1 if on else 0), "const_profile_enable")


def const_profile_read() -> Dict[str, Tuple[int, float]]:
    """kernel name -> (launches, total milliseconds) recorded since const_profile_enable(True)."""
    lib = load_library()
    cap = 64
    names = ctypes.create_string_buffer(4096)
    launches = (ctypes.c_int64 * cap)()
    ms = (ctypes.c_double * cap)()
    n = ctypes.c_int()
    _check(lib.const_profile_read(names, 4096, launches, ms, cap, ctypes.byref(n)), "const_profile_read")
    keys = [k for k in names.value.decode().split("\n") if k]
    return {k: (int(launches[i]), float(ms[i])) for i, k in enumerate(keys[:cap])}
