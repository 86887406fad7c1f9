"""Contraction oracle: Python front end.  TEST INFRASTRUCTURE ONLY (see package docstring).

Two evaluators of the same definition (paper Sec. 2.1, "Tensor contractions" / "Tensor
networks"; loop nest of Fig. 2(b)):

* `nary_direct` -- a generic, pure-Python evaluation of any product expression over sparse (COO)
  and dense operands: it enumerates every combination of stored nonzeros of the sparse operands
  whose shared indices agree, then every value of the indices that only dense operands carry,
  and adds the product into the output.  Exponential in spirit, for tiny inputs only.
* `ttmc3`, `ttmc4`, `mttkrp3`, `network` -- the same sums written as fixed loop nests in C
  (`contract_oracle.c`), in double precision, fast enough for millions of nonzeros.

Both return (S, A): the sum of the terms and the sum of their absolute values.
"""
from __future__ import annotations

import ctypes
import itertools
import re
from typing import Dict, List, Sequence, Tuple, Union

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_threads.argtypes = [ctypes.c_int]
        for name in ("oracle_ttmc3", "oracle_ttmc4", "oracle_mttkrp3", "oracle_network"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)     # exact widening for float32 inputs


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check_range(c: np.ndarray, extent: int, what: str) -> None:
    if c.size and (int(c.min()) < 0 or int(c.max()) >= extent):
        raise ValueError(f"coordinate out of range for {what}")


def _check_rc(rc: int) -> None:
    if rc == -2:
        raise ValueError("coordinate out of range")
    if rc != 0:
        raise MemoryError("oracle allocation failed")


def ttmc3(coords: Sequence[np.ndarray], vals, U, V, n_i: int) -> Tuple[np.ndarray, np.ndarray]:
    """Y[i,a,b] = sum_{j,k} X[i,j,k] U[j,a] V[k,b]  (Sec. 5.3)."""
    ci, cj, ck = (_i32(c) for c in coords)
    x, U, V = _f64(vals), _f64(U), _f64(V)
    _check_range(cj, U.shape[0], "j"); _check_range(ck, V.shape[0], "k")
    S = np.empty((n_i, U.shape[1], V.shape[1])); A = np.empty_like(S)
    c64 = ctypes.c_int64
    _check_rc(_load().oracle_ttmc3(c64(x.size), _p(ci), _p(cj), _p(ck), _p(x), _p(U), c64(U.shape[1]),
                                   _p(V), c64(V.shape[1]), c64(n_i), _p(S), _p(A)))
    return S, A


def ttmc4(coords, vals, U, V, W, n_i: int):
    """Y[i,a,b,c] = sum_{j,k,l} X[i,j,k,l] U[j,a] V[k,b] W[l,c]."""
    ci, cj, ck, cl = (_i32(c) for c in coords)
    x, U, V, W = _f64(vals), _f64(U), _f64(V), _f64(W)
    _check_range(cj, U.shape[0], "j"); _check_range(ck, V.shape[0], "k"); _check_range(cl, W.shape[0], "l")
    S = np.empty((n_i, U.shape[1], V.shape[1], W.shape[1])); A = np.empty_like(S)
    c64 = ctypes.c_int64
    _check_rc(_load().oracle_ttmc4(c64(x.size), _p(ci), _p(cj), _p(ck), _p(cl), _p(x), _p(U), c64(U.shape[1]),
                                   _p(V), c64(V.shape[1]), _p(W), c64(W.shape[1]), c64(n_i), _p(S), _p(A)))
    return S, A


def mttkrp3(coords, vals, B, C, n_i: int):
    """A[i,r] = sum_{j,k} X[i,j,k] B[j,r] C[k,r]  (Sec. 5.2)."""
    ci, cj, ck = (_i32(c) for c in coords)
    x, B, C = _f64(vals), _f64(B), _f64(C)
    if B.shape[1] != C.shape[1]:
        raise ValueError("rank mismatch")
    _check_range(cj, B.shape[0], "j"); _check_range(ck, C.shape[0], "k")
    S = np.empty((n_i, B.shape[1])); A = np.empty_like(S)
    c64 = ctypes.c_int64
    _check_rc(_load().oracle_mttkrp3(c64(x.size), _p(ci), _p(cj), _p(ck), _p(x), _p(B), _p(C),
                                     c64(B.shape[1]), c64(n_i), _p(S), _p(A)))
    return S, A


def network(u_coords, u_vals, V, w_coords, w_vals, n_i: int, n_k: int, n_m: int):
    """Z[i,m] = sum_{j,k,l} U[i,j,k] V[j,l] W[k,l,m]  (Sec. 1, second displayed equation)."""
    ui, uj, uk = (_i32(c) for c in u_coords)
    wk, wl, wm = (_i32(c) for c in w_coords)
    uv, wv, V = _f64(u_vals), _f64(w_vals), _f64(V)
    _check_range(uj, V.shape[0], "j"); _check_range(wl, V.shape[1], "l"); _check_range(wm, n_m, "m")
    S = np.empty((n_i, n_m)); A = np.empty_like(S)
    c64 = ctypes.c_int64
    _check_rc(_load().oracle_network(c64(uv.size), _p(ui), _p(uj), _p(uk), _p(uv), _p(V), c64(V.shape[1]),
                                     c64(wv.size), _p(wk), _p(wl), _p(wm), _p(wv),
                                     c64(n_i), c64(n_k), c64(n_m), _p(S), _p(A)))
    return S, A


# --------------------------------------------------------------------------------------
# generic direct n-ary evaluation (tiny inputs)
# --------------------------------------------------------------------------------------

_REF = re.compile(r"\s*([A-Za-z_][A-Za-z_0-9]*)\s*\[([^\]]*)\]\s*")

SparseArg = Tuple[Sequence[np.ndarray], np.ndarray]      # (coords per mode, values)


def _parse(expression: str):
    lhs, rhs = expression.split("=")
    def ref(text):
        m = _REF.fullmatch(text)
        if not m:
            raise ValueError(f"bad tensor reference: {text!r}")
        return m.group(1), [s.strip() for s in m.group(2).split(",") if s.strip()]
    return ref(lhs), [ref(t) for t in rhs.split("*")]


def nary_direct(expression: str, operands: Dict[str, Union[np.ndarray, SparseArg]],
                extents: Dict[str, int]) -> Tuple[np.ndarray, np.ndarray]:
    """Direct evaluation of `Out[...] = T1[...] * T2[...] * ...` from its definition.

    A dense operand is an ndarray; a sparse operand is (coords, vals) in COO form with
    coords[m] the coordinates of the m-th index of its reference.  Everything is widened to
    double.  For each binding of all indices that every sparse operand stores, the product of
    the operand values is added to Out at the external indices (Fig. 2(b), restricted to nz).
    """
    (out_name, out_idx), refs = _parse(expression)
    S = np.zeros([extents[i] for i in out_idx], dtype=np.float64)
    A = np.zeros_like(S)
    sparse_refs = [(n, idx) for n, idx in refs if not isinstance(operands[n], np.ndarray)]
    dense_refs = [(n, idx) for n, idx in refs if isinstance(operands[n], np.ndarray)]
    bound_by_sparse = []
    for _, idx in sparse_refs:
        for i in idx:
            if i not in bound_by_sparse:
                bound_by_sparse.append(i)
    all_idx = list(bound_by_sparse)
    for _, idx in dense_refs + [(out_name, out_idx)]:
        for i in idx:
            if i not in all_idx:
                all_idx.append(i)
    free_idx = [i for i in all_idx if i not in bound_by_sparse]

    def rec(level: int, binding: Dict[str, int], prod: float):
        if level == len(sparse_refs):
            for combo in itertools.product(*[range(extents[i]) for i in free_idx]):
                b = dict(binding)
                b.update(zip(free_idx, combo))
                term = prod
                for n, idx in dense_refs:
                    term *= float(operands[n][tuple(b[i] for i in idx)])
                o = tuple(b[i] for i in out_idx)
                S[o] += term
                A[o] += abs(term)
            return
        name, idx = sparse_refs[level]
        coords, vals = operands[name]
        for e in range(len(vals)):
            b = dict(binding)
            ok = True
            for m, i in enumerate(idx):
                c = int(coords[m][e])
                if i in b and b[i] != c:
                    ok = False
                    break
                b[i] = c
            if ok:
                rec(level + 1, b, prod * float(vals[e]))

    rec(0, {}, 1.0)
    return S, A


def nary_einsum(expression: str, operands: Dict[str, Union[np.ndarray, SparseArg]],
                extents: Dict[str, int]) -> Tuple[np.ndarray, np.ndarray]:
    """The same definition as `nary_direct` for inputs a Python loop nest cannot finish: every sparse
    operand is written out as a dense array (zeros where nothing is stored) and the sum over all index
    values of the product of the operands (Sec. 2.1, "Tensor networks") is taken by numpy.einsum in double
    precision, once on the values (S) and once on their absolute values (A = sum of |terms|, since the
    absolute value of a product is the product of the absolute values).  The index space must be small
    enough to enumerate (product of all extents up to ~1e8)."""
    (out_name, out_idx), refs = _parse(expression)
    letters = {}
    for _, idx in refs + [(out_name, out_idx)]:
        for i in idx:
            letters.setdefault(i, chr(ord("a") + len(letters)))
    dense = []
    for name, idx in refs:
        op = operands[name]
        if isinstance(op, np.ndarray):
            arr = np.asarray(op, dtype=np.float64)
        else:
            coords, vals = op
            arr = np.zeros([extents[i] for i in idx], dtype=np.float64)
            arr[tuple(np.asarray(c, dtype=np.int64) for c in coords)] = np.asarray(vals, dtype=np.float64)
        if arr.shape != tuple(extents[i] for i in idx):
            raise ValueError(f"operand {name} has shape {arr.shape}, expected {[extents[i] for i in idx]}")
        dense.append(arr)
    spec = ",".join("".join(letters[i] for i in idx) for _, idx in refs) + "->" + "".join(letters[i] for i in out_idx)
    S = np.einsum(spec, *dense, optimize=False)
    A = np.einsum(spec, *[np.abs(a) for a in dense], optimize=False)
    return np.ascontiguousarray(S), np.ascontiguousarray(A)
