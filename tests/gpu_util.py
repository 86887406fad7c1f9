"""Shared helpers of the GPU parity tests: run a workload through the C-ABI binding, run the oracle."""
import numpy as np
import torch

import paper_2401_04836_b200 as cb
from oracle import contract as oc
from oracle import csf as ocsf
from oracle import workload as ow

TOL = {np.dtype(np.float32): 1e-5, np.dtype(np.float64): 1e-12}    # |gpu - S| <= TOL * A per element


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def build_csf(op, mode_order):
    coords = [to_dev(c.astype(np.int32)) for c in op.coords]
    return cb.const_csf_build(coords, to_dev(op.vals), op.dims, mode_order)


def csf_to_host(h):
    pos, crd = [], []
    for l in range(h.order):
        p, c = cb.const_csf_level(h, l)
        pos.append(p.cpu().numpy())
        crd.append(c.cpu().numpy())
    return pos, crd, cb.const_csf_values(h).cpu().numpy()


def assert_csf_equal(h, op, mode_order):
    """Bit-exact comparison of every CSF array with the oracle's."""
    pos, crd, vals = csf_to_host(h)
    opos, ocrd, ovals = ocsf.build(op.coords, op.vals, mode_order)
    for l in range(len(mode_order)):
        np.testing.assert_array_equal(crd[l], ocrd[l], err_msg=f"crd level {l}")
        np.testing.assert_array_equal(pos[l], opos[l], err_msg=f"pos level {l}")
    assert vals.dtype == ovals.dtype and vals.tobytes() == ovals.tobytes()


def run_workload(w, bins=None, handles=None, tensor_stage=None):
    """Build CSF (unless given), create the plan, execute; returns (output ndarray, csf handles)."""
    dtype = cb.F32 if w.dtype == np.float32 else cb.F64
    if handles is None:
        handles = {n: build_csf(op, w.mode_orders[n]) for n, op in w.sparse.items()}
    if bins is not None:
        for h in handles.values():
            cb.const_csf_set_bins(h, *bins)
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, dtype)
    if tensor_stage is not None:
        cb.const_plan_set_tensor_stage(plan, tensor_stage)
    operands = dict(handles)
    operands.update({n: to_dev(a) for n, a in w.dense.items()})
    out = torch.full(w.out_shape, float("nan"), dtype=torch.float32 if dtype == cb.F32 else torch.float64,
                     device="cuda")                               # the library must overwrite every element
    cb.const_execute(plan, operands, out)
    assert cb.const_last_device_status(plan) == 0
    return out.cpu().numpy(), handles


def oracle(w, rows=None):
    """(S, A) of the workload's expression; rows = only these output rows (others are returned as zeros)."""
    return ow.evaluate(w, rows)


def assert_close(out, S, A, dtype, rows=None):
    tol = TOL[np.dtype(dtype)]
    if rows is not None:
        out, S, A = out[rows], S[rows], A[rows]
    assert np.all(np.isfinite(out)), "output holds NaN/Inf (an element was never written?)"
    err = np.abs(out.astype(np.float64) - S)
    bound = tol * A
    bad = err > bound
    if bad.any():
        worst = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{bad.sum()} elements beyond {tol} * sum|terms|; worst at {worst}: "
                             f"gpu={out[worst]!r} oracle={S[worst]!r} sum|terms|={A[worst]!r}")
    return float(np.max(err / np.maximum(bound, 1e-300)))
