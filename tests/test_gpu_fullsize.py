"""The five benchmark configurations at full size, in the launch configuration bench.py times.

  * CSF: the oracle cannot sort 10^8 nonzeros in seconds, so the arrays are checked by properties
    that hold at any size (level sizes against distinct-prefix counts computed on the host; pos/crd
    invariants over the whole arrays) and, for sampled root slices (the largest and the smallest
    included), every array segment bit-exact against the CSF oracle built from that slice alone;
  * contraction: EVERY output row, element by element, against the fp64 oracle evaluated on the whole
    tensor (|gpu - S| <= tol * sum|terms|, and exactly 0 where no term exists).  The oracle result of a
    configuration is computed once and shared by the parametrisations that use it.
"""
import functools

import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from oracle import csf as ocsf
from workloads import make_config, row_sample
from tests.gpu_util import assert_close, build_csf, oracle, to_dev

pytestmark = pytest.mark.gpu


def _sample_rows(op, mode, n_random, rng):
    sizes = np.bincount(op.coords[mode], minlength=op.dims[mode])
    present = np.nonzero(sizes)[0]
    rows = set(rng.choice(present, size=min(n_random, present.size), replace=False).tolist())
    rows.add(int(np.argmax(sizes)))                          # the largest slice
    rows.add(int(present[np.argmin(sizes[present])]))        # and the smallest
    return np.array(sorted(rows))


def _check_csf(h, op, mode_order, rows):
    order = len(mode_order)
    lev = [op.coords[m] for m in mode_order]
    pos, crd = [], []
    for l in range(order):
        p, c = cb.const_csf_level(h, l)
        pos.append(p)
        crd.append(c)
    vals = cb.const_csf_values(h)
    # level sizes = number of distinct prefixes
    key = np.zeros(op.nnz, dtype=np.uint64)
    for l in range(order - 1):
        key = key * np.uint64(op.dims[mode_order[l]]) + lev[l].astype(np.uint64)
        assert crd[l].numel() == np.unique(key).size, f"size of level {l}"
    assert crd[order - 1].numel() == op.nnz and vals.numel() == op.nnz
    # structural invariants over the whole arrays (on the device)
    assert pos[0].tolist() == [0, crd[0].numel()]
    for l in range(1, order):
        p = pos[l]
        assert p.numel() == crd[l - 1].numel() + 1 and int(p[0]) == 0 and int(p[-1]) == crd[l].numel()
        assert bool((p[1:] > p[:-1]).all()), f"pos level {l} must increase strictly (no empty node)"
    for l in range(order):
        c = crd[l]
        assert int(c.min()) >= 0 and int(c.max()) < op.dims[mode_order[l]]
        inc = torch.ones(c.numel(), dtype=torch.bool, device=c.device)
        inc[1:] = c[1:] > c[:-1]
        starts = pos[l][:-1].long() if l > 0 else torch.zeros(1, dtype=torch.long, device=c.device)
        inc[starts] = True                                    # the first child of a parent may restart
        assert bool(inc.all()), f"crd level {l} must increase inside every parent"
    # sampled slices: every segment bit-exact against the oracle built from the slice alone
    crd0 = crd[0].cpu().numpy()
    for r in rows:
        sub = row_sample(op, [r], mode=mode_order[0])
        opos, ocrd, ovals = ocsf.build(sub.coords, sub.vals, mode_order)
        s = int(np.searchsorted(crd0, r))
        assert crd0[s] == r
        lo, hi = s, s + 1
        for l in range(1, order):
            seg_pos = pos[l][lo:hi + 1].cpu().numpy()
            np.testing.assert_array_equal(seg_pos - seg_pos[0], opos[l], err_msg=f"pos level {l}, slice {r}")
            lo, hi = int(seg_pos[0]), int(seg_pos[-1])
            np.testing.assert_array_equal(crd[l][lo:hi].cpu().numpy(), ocrd[l], err_msg=f"crd level {l}, slice {r}")
        assert vals[lo:hi].cpu().numpy().tobytes() == ovals.tobytes(), f"values of slice {r}"


@functools.lru_cache(maxsize=None)
def _workload(config_id):
    return make_config(config_id)


@functools.lru_cache(maxsize=None)
def _oracle_all_rows(config_id):
    """(S, A) over every output row: tens of seconds of host time per configuration."""
    return oracle(_workload(config_id))


@pytest.mark.parametrize("config_id,tensor_stage", [(2, None), (2, True), (3, False), (3, True), (4, None), (5, None)])
def test_full_size_config(config_id, tensor_stage):
    rng = np.random.default_rng(100 + config_id)
    w = _workload(config_id)
    dtype = cb.F32 if w.dtype == np.float32 else cb.F64
    handles = {}
    for name, op in w.sparse.items():
        mo = w.mode_orders[name]
        handles[name] = build_csf(op, mo)
        rows_csf = _sample_rows(op, mo[0], 6, rng)
        _check_csf(handles[name], op, mo, rows_csf)
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, dtype)
    if tensor_stage is not None:
        cb.const_plan_set_tensor_stage(plan, tensor_stage)     # TTMc: per-slice stage on tensor cores or FMA pipes
    operands = dict(handles)
    operands.update({n: to_dev(a) for n, a in w.dense.items()})
    out = torch.full(w.out_shape, float("nan"), dtype=torch.float32 if dtype == cb.F32 else torch.float64,
                     device="cuda")
    cb.const_execute(plan, operands, out)
    assert cb.const_last_device_status(plan) == 0
    out = out.cpu().numpy()
    # the default thresholds put slices of this tensor into every bin the family uses, and every row is compared
    first = w.sparse["U" if w.family == "network" else "X"]
    if w.family != "network":
        counts = cb.const_csf_bin_counts(handles["X"])
        assert counts["light"] > 0 and counts["heavy"] > 0 and counts["giant"] > 0, counts
    S, A = _oracle_all_rows(config_id)
    assert_close(out, S, A, w.dtype)
    # rows whose slice is empty stay exactly zero
    empty = np.setdiff1d(np.arange(first.dims[0]), first.coords[0])
    assert np.all(out[empty] == 0)
