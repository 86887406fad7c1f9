"""The generic executor (loop tree of Sec. 4.2 walked on the GPU) against the oracle.

Schedules no hand-written kernel family covers -- the four-tensor running example with the schedule the
paper prints (Fig. 5), order-4 MTTKRP, TTMc at other ranks and in fp64, the two-contraction network in its
scatter form and unfused, a network multiplied by a sparse 0/1 map (Sec. 5.1, Eq. 2) -- and, through
const_plan_set_generic_executor, schedules the families do cover.  Element by element:
|gpu - S| <= tol * sum|terms|, exact zeros where no term exists.
"""
import json
import os

import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from oracle import contract as oc
from workloads import make_config, network_workload, ttmc3_workload, ttmc4_workload, mttkrp_workload
from workloads import generators as gen
from tests.gpu_util import assert_close, build_csf, oracle, to_dev

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
NP = {cb.F32: np.float32, cb.F64: np.float64}


def sparse_input(rng, dims, nnz, dtype):
    return gen._uniform_tensor(dims, nnz, rng, "pm1", dtype)


def run_tree(expression, tree, mode_orders, loop_orders, extents, dtype, sparse, dense, out_shape, generic=None):
    """Build every CSF operand with its mode order, create the plan, execute; returns (output, family)."""
    plan = cb.const_plan_create(expression, tree, mode_orders, loop_orders, extents, dtype)
    if generic is not None:
        cb.const_plan_set_generic_executor(plan, generic)
    ops = {n: build_csf(op, mode_orders[n]) for n, op in sparse.items()}
    ops.update({n: to_dev(a) for n, a in dense.items()})
    out = torch.full(out_shape, float("nan"), dtype=torch.float32 if dtype == cb.F32 else torch.float64, device="cuda")
    cb.const_execute(plan, ops, out)
    assert cb.const_last_device_status(plan) == 0
    return out.cpu().numpy(), cb.const_plan_family(plan)


def coo(op):
    return (op.coords, op.vals)


@pytest.mark.parametrize("dtype", [cb.F64, cb.F32])
@pytest.mark.parametrize("n,nnz", [(4, 20), (14, 300)])
def test_running_example_with_the_printed_schedule(dtype, n, nnz):
    """R_ijk = A_ipq B_jpr C_kqr D_jkr, tree X = A B, Y = X C, R = Y D, all four inputs in CSF with the mode
    orders of Fig. 5, loops r, j fused so that X and Y are 2-D workspaces."""
    with open(os.path.join(GOLDEN, "running_example_schedule.json")) as f:
        g = json.load(f)
    rng = np.random.default_rng(1000 * n + dtype)
    ext = {"i": n, "j": n + 1, "k": n + 2, "p": n, "q": n + 3, "r": n - 1}
    shape = {"A": "ipq", "B": "jpr", "C": "kqr", "D": "jkr"}
    sparse = {t: sparse_input(rng, tuple(ext[x] for x in idx), nnz, NP[dtype]) for t, idx in shape.items()}
    out, family = run_tree(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], ext, dtype, sparse, {},
                           (ext["i"], ext["j"], ext["k"]))
    assert family == "tree"
    ops = {t: coo(op) for t, op in sparse.items()}
    S, A = (oc.nary_direct if n <= 4 else oc.nary_einsum)(g["expression"], ops, ext)
    assert np.count_nonzero(A) > 0
    assert_close(out, S, A, NP[dtype])


def test_running_example_other_legal_schedules():
    """The same network with the first contraction in a nest of its own, and fused on r only."""
    rng = np.random.default_rng(77)
    ext = {"i": 6, "j": 7, "k": 5, "p": 6, "q": 4, "r": 5}
    shape = {"A": "ipq", "B": "jpr", "C": "kqr", "D": "jkr"}
    sparse = {t: sparse_input(rng, tuple(ext[x] for x in idx), 60, np.float64) for t, idx in shape.items()}
    expr = "R[i,j,k] = A[i,p,q] * B[j,p,r] * C[k,q,r] * D[j,k,r]"
    tree = ["X[i,j,q,r] = A[i,p,q] * B[j,p,r]", "Y[i,j,k,r] = X[i,j,q,r] * C[k,q,r]", "R[i,j,k] = Y[i,j,k,r] * D[j,k,r]"]
    S, A = oc.nary_einsum(expr, {t: coo(op) for t, op in sparse.items()}, ext)
    mo = {"A": [1, 2, 0], "B": [2, 0, 1], "C": [2, 1, 0], "D": [2, 0, 1]}
    for loops in (["rjpqi", "irqkj", "irjk"],          # X is a full-order global workspace; Y is fused on i and r
                  ["rjpqi", "rqkji", "rjki"]):         # only r is shared by all three
        out, family = run_tree(expr, tree, mo, loops, ext, cb.F64, sparse, {}, (6, 7, 5))
        assert family == "tree"
        assert_close(out, S, A, np.float64)


def test_generic_executor_on_schedules_the_families_cover():
    w = make_config(1)
    S, A = oracle(w)
    out, family = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32, w.sparse, w.dense,
                           w.out_shape, generic=True)
    assert family == "ttmc3"
    assert_close(out, S, A, np.float32)
    w = mttkrp_workload((40, 35, 30), 3_000, 8, slice_s=1.2, value="unit", config_id=4)
    S, A = oracle(w)
    out, _ = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32, w.sparse, w.dense,
                      w.out_shape, generic=True)
    assert_close(out, S, A, np.float32)
    w = network_workload(32, 8, 4, 0.3, config_id=5)
    S, A = oracle(w)
    out, _ = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F64, w.sparse, w.dense,
                      w.out_shape, generic=True)
    assert_close(out, S, A, np.float64)


@pytest.mark.parametrize("rank", [4, 12, 16])
def test_ttmc4_at_ranks_without_a_hand_written_kernel(rank):
    w = ttmc4_workload((30, 12, 10, 9), 2_500, rank, slice_s=1.0, value="pm1", config_id=3)
    out, family = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32, w.sparse, w.dense,
                           w.out_shape)
    assert family == "tree"
    S, A = oracle(w)
    assert_close(out, S, A, np.float32)


def test_ttmc3_in_fp64_and_with_an_unfused_consumer():
    w = ttmc3_workload((25, 20, 30), 1_500, (6, 10), value="pm1", config_id=31)
    X = w.sparse["X"]
    X64 = gen.SparseOperand(X.coords, X.vals.astype(np.float64), X.dims)
    dense = {n: a.astype(np.float64) for n, a in w.dense.items()}
    S, A = oc.ttmc3(X.coords, X64.vals, dense["U"], dense["V"], X.dims[0])
    for loops in (w.loop_orders, ["ijkb", "iajb"]):              # t[b] per (i,j); or t[j,b] per i with a, j swapped
        out, family = run_tree(w.expression, w.tree, w.mode_orders, loops, w.extents, cb.F64, {"X": X64}, dense,
                               w.out_shape)
        assert family == "tree"
        assert_close(out, S, A, np.float64)


def test_order4_mttkrp():
    rng = np.random.default_rng(41)
    dims, r = (20, 9, 8, 7), 5
    X = sparse_input(rng, dims, 900, np.float32)
    fac = {n: rng.standard_normal((d, r)).astype(np.float32) for n, d in zip("BCD", dims[1:])}
    expr = "M[i,r] = X[i,j,k,l] * B[j,r] * C[k,r] * D[l,r]"
    tree = ["P[i,j,k,r] = X[i,j,k,l] * D[l,r]", "Q[i,j,r] = P[i,j,k,r] * C[k,r]", "M[i,r] = Q[i,j,r] * B[j,r]"]
    ext = {"i": 20, "j": 9, "k": 8, "l": 7, "r": r}
    out, family = run_tree(expr, tree, {"X": (0, 1, 2, 3)}, ["ijklr", "ijkr", "ijr"], ext, cb.F32, {"X": X}, fac, (20, r))
    assert family == "tree"
    S, A = oc.nary_einsum(expr, dict(fac, X=coo(X)), ext)
    assert_close(out, S, A, np.float32)


def test_network_scatter_form_and_unfused():
    """Z_im = U_ijk V_jl W_klm with U stored (i,j,k) and W stored (k,l,m): both contractions scatter into the
    workspace; and the gather-form mode orders with the two contractions not fused at all."""
    w = network_workload(24, 6, 4, 0.3, config_id=51)
    S, A = oracle(w)
    out, family = run_tree(w.expression, w.tree, {"U": (0, 1, 2), "W": (0, 1, 2)}, ["ijkl", "iklm"], w.extents, cb.F64,
                           w.sparse, w.dense, w.out_shape)
    assert family == "tree"
    assert_close(out, S, A, np.float64)
    out, family = run_tree(w.expression, w.tree, w.mode_orders, ["ikjl", "lmik"], w.extents, cb.F64, w.sparse, w.dense,
                           w.out_shape)
    assert family == "tree"
    assert_close(out, S, A, np.float64)


@pytest.mark.parametrize("sparse_c", [False, True])
def test_network_restricted_by_a_sparse_map(sparse_c):
    """E_{K i m} = I_{K u v} C_{u i} P_{v m} L_{K i} with L a 0/1 sparse map (Sec. 5.1, Eq. 2): the loops over
    K and i are fused and follow the map, so nothing outside it is evaluated."""
    rng = np.random.default_rng(52 + sparse_c)
    ext = {"k": 18, "u": 12, "v": 10, "i": 9, "m": 11}
    I3 = sparse_input(rng, (18, 12, 10), 400, np.float64)
    L = sparse_input(rng, (18, 9), 50, np.float64)
    L = gen.SparseOperand(L.coords, np.ones_like(L.vals), L.dims)
    P = rng.standard_normal((10, 11))
    expr = "E[k,i,m] = I[k,u,v] * C[u,i] * P[v,m] * L[k,i]"
    tree = ["S[k,v,i] = I[k,u,v] * C[u,i]", "T[k,i,m] = S[k,v,i] * P[v,m]", "E[k,i,m] = T[k,i,m] * L[k,i]"]
    loops = ["kiuv", "kivm", "kim"]
    if sparse_c:
        C = sparse_input(rng, (12, 9), 60, np.float64)
        sparse, dense = {"I": I3, "C": C, "L": L}, {"P": P}
        mo = {"I": (0, 1, 2), "C": (1, 0), "L": (0, 1)}         # C stored (i, u): i is bound before u
        ops = {"I": coo(I3), "C": coo(C), "P": P, "L": coo(L)}
    else:
        C = rng.standard_normal((12, 9))
        sparse, dense = {"I": I3, "L": L}, {"C": C, "P": P}
        mo = {"I": (0, 1, 2), "L": (0, 1)}
        ops = {"I": coo(I3), "C": C, "P": P, "L": coo(L)}
    out, family = run_tree(expr, tree, mo, loops, ext, cb.F64, sparse, dense, (18, 9, 11))
    assert family == "tree"
    S, A = oc.nary_einsum(expr, ops, ext)
    assert_close(out, S, A, np.float64)
    mask = np.zeros((18, 9), bool)
    mask[L.coords[0], L.coords[1]] = True
    assert np.all(out[~mask] == 0) and np.count_nonzero(out[mask]) > 0


def test_empty_operand_and_operand_checks():
    w = ttmc3_workload((6, 5, 4), 10, (3, 5), value="pm1", config_id=32)
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    assert cb.const_plan_family(plan) == "tree"
    empty = gen.SparseOperand([np.zeros(0, np.int32)] * 3, np.zeros(0, np.float32), (6, 5, 4))
    out = torch.full(w.out_shape, float("nan"), device="cuda")
    cb.const_execute(plan, {"X": build_csf(empty, (0, 1, 2)), "U": to_dev(w.dense["U"]), "V": to_dev(w.dense["V"])}, out)
    assert np.all(out.cpu().numpy() == 0)
    with pytest.raises(cb.ConstError):
        cb.const_execute(plan, {"X": build_csf(w.sparse["X"], (1, 0, 2)), "U": to_dev(w.dense["U"]),
                                "V": to_dev(w.dense["V"])}, out)         # CSF built with another mode order
    with pytest.raises(cb.ConstError):
        cb.const_execute(plan, {"X": build_csf(w.sparse["X"], (0, 1, 2)), "U": to_dev(w.dense["U"])}, out)
    with pytest.raises(cb.ConstError):
        cb.const_plan_set_generic_executor(plan, False)                  # this plan has no other kernel


def test_random_legal_schedules_of_the_running_example():
    """Sixty seeded schedules of R_ijk = A_ipq B_jpr C_kqr D_jkr: random loop permutations per contraction (half of
    them forced to share leading loops, so that fused nests with reduced workspaces come up as often as plain
    ones), every CSF operand stored in the mode order its reader's loops ask for (Sec. 3.2).  Whatever the checker
    accepts must run and give the one result the expression defines."""
    rng = np.random.default_rng(2401)
    ext = {"i": 6, "j": 7, "k": 5, "p": 6, "q": 4, "r": 5}
    shape = {"A": "ipq", "B": "jpr", "C": "kqr", "D": "jkr"}
    reader = {"A": 0, "B": 0, "C": 1, "D": 2}
    sparse = {t: sparse_input(rng, tuple(ext[x] for x in idx), 70, np.float64) for t, idx in shape.items()}
    expr = "R[i,j,k] = A[i,p,q] * B[j,p,r] * C[k,q,r] * D[j,k,r]"
    tree = ["X[i,j,q,r] = A[i,p,q] * B[j,p,r]", "Y[i,j,k,r] = X[i,j,q,r] * C[k,q,r]", "R[i,j,k] = Y[i,j,k,r] * D[j,k,r]"]
    S, A = oc.nary_einsum(expr, {t: coo(op) for t, op in sparse.items()}, ext)
    ran, fused = 0, 0
    for trial in range(60):
        loops = []
        lead = "".join(rng.permutation(list("ijr")))[: int(rng.integers(1, 4))] if trial % 2 else ""
        for idx in ("ijpqr", "ijkqr", "ijkr"):
            rest = [c for c in idx if c not in lead]
            loops.append(lead + "".join(rng.permutation(rest)))
        mo = {n: [int(x) for x in np.argsort([loops[reader[n]].index(c) for c in shape[n]])] for n in shape}
        try:
            plan = cb.const_plan_create(expr, tree, mo, loops, ext, cb.F64)
        except cb.ConstError as e:
            assert e.status == 3, (loops, e.status)              # an illegal schedule is the only reason to refuse
            continue
        text = cb.const_plan_describe(plan)
        fused += "zero " in text
        out, family = run_tree(expr, tree, mo, loops, ext, cb.F64, sparse, {}, (6, 7, 5))
        assert family == "tree"
        assert_close(out, S, A, np.float64)
        ran += 1
    assert ran >= 40 and fused >= 10, (ran, fused)


@pytest.mark.parametrize("dtype", [cb.F64, cb.F32])
def test_every_tree_of_the_network_under_random_schedules(dtype):
    """Z_im = U_ijk V_jl W_klm (Sec. 1) through each of its three contraction trees -- (U V) W, U (V W) and
    (U W) V -- with ninety seeded loop orders, half of them sharing leading loops so that the intermediate loses
    modes.  All trees and all schedules define the same Z."""
    rng = np.random.default_rng(4836)
    ext = {"i": 9, "j": 7, "k": 8, "l": 5, "m": 6}
    shape = {"U": "ijk", "W": "klm"}
    sparse = {t: sparse_input(rng, tuple(ext[x] for x in idx), 90, NP[dtype]) for t, idx in shape.items()}
    V = rng.uniform(-1.0, 1.0, (ext["j"], ext["l"])).astype(NP[dtype])
    expr = "Z[i,m] = U[i,j,k] * V[j,l] * W[k,l,m]"
    trees = [(["T[i,k,l] = U[i,j,k] * V[j,l]", "Z[i,m] = T[i,k,l] * W[k,l,m]"], ("ijkl", "iklm"), {"U": 0, "W": 1}),
             (["T[j,k,m] = V[j,l] * W[k,l,m]", "Z[i,m] = U[i,j,k] * T[j,k,m]"], ("jklm", "ijkm"), {"U": 1, "W": 0}),
             (["T[i,j,l,m] = U[i,j,k] * W[k,l,m]", "Z[i,m] = T[i,j,l,m] * V[j,l]"], ("ijklm", "ijlm"), {"U": 0, "W": 0})]
    ops = {t: coo(op) for t, op in sparse.items()}
    ops["V"] = V
    S, A = oc.nary_einsum(expr, ops, ext)
    fused = 0
    for trial in range(90):
        tree, idxs, reader = trees[trial % 3]
        shared = [c for c in idxs[0] if c in idxs[1]]
        lead = "".join(rng.permutation(shared))[: int(rng.integers(0, len(shared) + 1))] if trial % 2 else ""
        loops = [lead + "".join(rng.permutation([c for c in s if c not in lead])) for s in idxs]
        mo = {n: [int(x) for x in np.argsort([loops[reader[n]].index(c) for c in shape[n]])] for n in shape}
        plan = cb.const_plan_create(expr, tree, mo, loops, ext, dtype)
        fused += "zero " in cb.const_plan_describe(plan)
        out, _ = run_tree(expr, tree, mo, loops, ext, dtype, sparse, {"V": V}, (ext["i"], ext["m"]), generic=True)
        assert_close(out, S, A, NP[dtype])
    assert fused >= 20, fused


def test_medium_sizes_reach_every_way_the_iterations_are_dealt_out():
    """Sizes at which the executor's launch logic leaves its small-case settings: (a) 400 K nonzeros in about as
    many (i, j) fibres with a 12-element workspace -- one fibre per warp, runs of several consecutive fibres per
    warp, the slice above a fibre followed along the run; (b) fp64 workspaces of 4.8 KB -- one fibre per block,
    workspaces in shared memory; (c) a 122 KB workspace per outer iteration -- workspaces in global scratch."""
    w = ttmc3_workload((4000, 300, 400), 400_000, (12, 12), slice_s=1.1, value="pm1", config_id=61)
    S, A = oracle(w)
    out, family = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32, w.sparse, w.dense,
                           w.out_shape)
    assert family == "tree"
    assert_close(out, S, A, np.float32)

    w = ttmc4_workload((300, 100, 20, 20), 60_000, 24, slice_s=1.0, value="pm1", config_id=62)
    X = w.sparse["X"]
    sparse = {"X": gen.SparseOperand(X.coords, X.vals.astype(np.float64), X.dims)}
    dense = {n: a.astype(np.float64) for n, a in w.dense.items()}
    S, A = oracle(w)                                              # fp64 throughout; the inputs are fp32 values
    out, family = run_tree(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F64, sparse, dense,
                           w.out_shape)
    assert family == "tree"
    assert_close(out, S, A, np.float64)

    w = network_workload(160, 96, 8, 0.3, config_id=63)
    S, A = oracle(w)
    out, family = run_tree(w.expression, w.tree, {"U": (0, 1, 2), "W": (0, 1, 2)}, ["ijkl", "iklm"], w.extents, cb.F64,
                           w.sparse, w.dense, w.out_shape)
    assert family == "tree"
    assert_close(out, S, A, np.float64)


def test_running_example_degenerate_operands():
    """Each of the four operands empty in turn (the result is exactly zero whichever loop walks or looks up the
    empty tensor), and every extent equal to one (a single product)."""
    with open(os.path.join(GOLDEN, "running_example_schedule.json")) as f:
        g = json.load(f)
    rng = np.random.default_rng(99)
    ext = {"i": 5, "j": 6, "k": 4, "p": 5, "q": 3, "r": 4}
    shape = {"A": "ipq", "B": "jpr", "C": "kqr", "D": "jkr"}
    full = {t: sparse_input(rng, tuple(ext[x] for x in idx), 40, np.float64) for t, idx in shape.items()}
    for hollow in shape:
        dims = tuple(ext[x] for x in shape[hollow])
        sparse = dict(full)
        sparse[hollow] = gen.SparseOperand([np.zeros(0, np.int32)] * 3, np.zeros(0, np.float64), dims)
        out, _ = run_tree(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], ext, cb.F64, sparse, {},
                          (ext["i"], ext["j"], ext["k"]))
        assert np.array_equal(out, np.zeros_like(out)), hollow
    one = {x: 1 for x in ext}
    vals = {"A": 1.5, "B": -2.0, "C": 0.25, "D": 3.0}
    sparse = {t: gen.SparseOperand([np.zeros(1, np.int32)] * 3, np.array([v]), (1, 1, 1)) for t, v in vals.items()}
    out, _ = run_tree(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], one, cb.F64, sparse, {}, (1, 1, 1))
    assert out.tolist() == [[[1.5 * -2.0 * 0.25 * 3.0]]]
