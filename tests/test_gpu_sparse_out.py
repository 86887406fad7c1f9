"""Results in CSF form (const_csf_from_dense) and the 4-index contraction of Sec. 5.1, Eq. 3.

  * conversion: every CSF array bit-exact against the CSF oracle built from the array's nonzero entries;
  * V_{i j m n} = E_{K i m} E_{K j n} (Eq. 3) with both operands in CSF form obtained from a dense E, on the
    generic executor, element by element against the oracle;
  * a network restricted by a sparse map (Eq. 2), its dense result converted to CSF: the stored pattern is the
    set of entries that have terms, the stored values meet the tolerance.
"""
import itertools

import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from oracle import contract as oc
from oracle import csf as ocsf
from workloads import generators as gen
from tests.gpu_util import TOL, assert_close, build_csf, csf_to_host, to_dev

pytestmark = pytest.mark.gpu


def sparse_dense_array(rng, shape, density, dtype):
    a = rng.standard_normal(shape).astype(dtype)
    a[rng.random(shape) >= density] = 0
    return a


def coo_of(a):
    coords = np.nonzero(a)
    return [c.astype(np.int32) for c in coords], a[coords]


@pytest.mark.parametrize("shape,dtype", [((37, 23), np.float32), ((9, 14, 11), np.float64), ((5, 6, 7, 4), np.float32),
                                         ((300, 41, 29), np.float32)])
def test_conversion_is_bit_exact(shape, dtype):
    rng = np.random.default_rng(len(shape) * 100 + shape[0])
    a = sparse_dense_array(rng, shape, 0.3, dtype)
    a.flat[3] = -0.0                                             # compares equal to zero: not stored
    coords, vals = coo_of(a)
    orders = list(itertools.permutations(range(len(shape))))
    for mo in orders[:: max(1, len(orders) // 4)]:
        h = cb.const_csf_from_dense(to_dev(a), mo)
        pos, crd, v = csf_to_host(h)
        opos, ocrd, ovals = ocsf.build(coords, vals, mo)
        for l in range(len(shape)):
            np.testing.assert_array_equal(crd[l], ocrd[l])
            np.testing.assert_array_equal(pos[l], opos[l])
        assert v.dtype == ovals.dtype and v.tobytes() == ovals.tobytes()
    h = cb.const_csf_from_dense(to_dev(np.zeros(shape, dtype)), orders[0])      # nothing stored at all
    assert all(c.size == 0 for c in csf_to_host(h)[1])


def test_four_index_contraction_from_csf_operands():
    rng = np.random.default_rng(63)
    ext = {"k": 16, "i": 9, "j": 9, "m": 7, "n": 7}
    E = sparse_dense_array(rng, (16, 9, 7), 0.25, np.float64)
    e1 = cb.const_csf_from_dense(to_dev(E), (0, 1, 2))
    e2 = cb.const_csf_from_dense(to_dev(E), (0, 1, 2))
    expr = "V[i,j,m,n] = A[k,i,m] * B[k,j,n]"
    plan = cb.const_plan_create(expr, [expr], {"A": (0, 1, 2), "B": (0, 1, 2)}, ["kimjn"], ext, cb.F64)
    assert cb.const_plan_family(plan) == "tree"
    out = torch.full((9, 9, 7, 7), float("nan"), dtype=torch.float64, device="cuda")
    cb.const_execute(plan, {"A": e1, "B": e2}, out)
    assert cb.const_last_device_status(plan) == 0
    S, A = oc.nary_einsum(expr, {"A": coo_of(E), "B": coo_of(E)}, ext)
    assert_close(out.cpu().numpy(), S, A, np.float64)
    # and the result itself as a CSF tensor: its pattern is where terms exist
    hv = cb.const_csf_from_dense(out, (0, 1, 2, 3))
    _, crd, vals = csf_to_host(hv)
    assert vals.size == np.count_nonzero(A)


def test_restricted_network_result_in_csf_form():
    rng = np.random.default_rng(64)
    ext = {"k": 14, "u": 10, "v": 9, "i": 8, "m": 6}
    I3 = gen._uniform_tensor((14, 10, 9), 300, rng, "pm1", np.float64)
    L = gen._uniform_tensor((14, 8), 40, rng, "pm1", np.float64)
    L = gen.SparseOperand(L.coords, np.ones_like(L.vals), L.dims)
    C, P = rng.standard_normal((10, 8)), rng.standard_normal((9, 6))
    expr = "E[k,i,m] = I[k,u,v] * C[u,i] * P[v,m] * L[k,i]"
    tree = ["S[k,v,i] = I[k,u,v] * C[u,i]", "T[k,i,m] = S[k,v,i] * P[v,m]", "E[k,i,m] = T[k,i,m] * L[k,i]"]
    plan = cb.const_plan_create(expr, tree, {"I": (0, 1, 2), "L": (0, 1)}, ["kiuv", "kivm", "kim"], ext, cb.F64)
    out = torch.full((14, 8, 6), float("nan"), dtype=torch.float64, device="cuda")
    cb.const_execute(plan, {"I": build_csf(I3, (0, 1, 2)), "L": build_csf(L, (0, 1)), "C": to_dev(C), "P": to_dev(P)}, out)
    S, A = oc.nary_einsum(expr, {"I": (I3.coords, I3.vals), "C": C, "P": P, "L": (L.coords, L.vals)}, ext)
    h = cb.const_csf_from_dense(out, (0, 1, 2))
    pos, crd, vals = csf_to_host(h)
    # expand the CSF back to coordinates (pure bookkeeping) and compare what is unique: the pattern, then the values
    k = np.repeat(crd[0], np.diff(pos[1]))
    ki = np.repeat(np.arange(crd[1].size), np.diff(pos[2]))
    kk, ii, mm = k[ki], crd[1][ki], crd[2]
    stored = np.zeros(S.shape, bool)
    stored[kk, ii, mm] = True
    np.testing.assert_array_equal(stored, A > 0)
    assert np.all(np.abs(vals - S[kk, ii, mm]) <= TOL[np.dtype(np.float64)] * A[kk, ii, mm])
