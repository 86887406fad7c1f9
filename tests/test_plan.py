"""Host-side schedule checker and kernel-family matcher (Sec. 3.2 constraints on a given solution)."""
import json
import os

import pytest

import paper_2401_04836_b200 as cb
from workloads import make_config, ttmc3_workload, ttmc4_workload, mttkrp_workload, network_workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _status(fn, *a, **k):
    try:
        fn(*a, **k)
        return 0
    except cb.ConstError as e:
        return e.status


def _running_example():
    with open(os.path.join(GOLDEN, "running_example_schedule.json")) as f:
        g = json.load(f)
    ext = {x: 5 for x in "ijkpqr"}
    return g, ext


def test_paper_running_example_is_legal_and_reduces_to_2d():
    """The constraint solution the paper prints (Fig. 5; dp_A = 2,0,1; lp_0 = r0 j1 p2 q3 i4) passes, and
    fusing r, j leaves X and Y as order-2 workspaces."""
    g, ext = _running_example()
    red = cb.const_schedule_check(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], ext)
    assert red == [g["reduced_orders"]["X"], g["reduced_orders"]["Y"], 0]
    # no hand-written kernel family matches four sparse tensors: the plan binds to the generic executor
    p = cb.const_plan_create(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], ext, cb.F64)
    assert cb.const_plan_family(p) == "tree"
    assert [cb.const_plan_reduced_order(p, c) for c in range(3)] == [2, 2, 0]


def test_paper_running_example_violations():
    g, ext = _running_example()
    chk = lambda **kw: _status(cb.const_schedule_check, kw.get("expression", g["expression"]),
                               kw.get("tree", g["tree"]), kw.get("mode_orders", g["mode_orders"]),
                               kw.get("loop_orders", g["loop_orders"]), ext)
    assert chk() == 0
    # Sec. 3.2.4: A is stored (p,q,i); a loop order with q before p cannot traverse it
    assert chk(loop_orders=["rjqpi", "rjqki", "rjki"]) == 3
    # the paper's worked pair (dp_A0 < dp_A2 => lp_i < lp_q): store A as (i,p,q) but keep loops r,j,p,q,i
    mo = dict(g["mode_orders"]); mo["A"] = [0, 1, 2]
    assert chk(mode_orders=mo) == 3
    # Sec. 3.2.1: child before parent
    assert chk(tree=[g["tree"][1], g["tree"][0], g["tree"][2]],
               loop_orders=[g["loop_orders"][1], g["loop_orders"][0], g["loop_orders"][2]]) == 3
    # Sec. 3.2.2 / 3.2.3: not permutations
    mo = dict(g["mode_orders"]); mo["B"] = [2, 2, 1]
    assert chk(mode_orders=mo) == 3
    assert chk(loop_orders=["rjpq", "rjqki", "rjki"]) == 3
    assert chk(loop_orders=["rjpqik", "rjqki", "rjki"]) == 3
    # an index of the result may not be summed; an index may not be summed while a tensor outside the
    # sub-tree still carries it (r occurs in C and D)
    assert chk(tree=["X[i,j,q] = A[i,p,q] * B[j,p,r]", "Y[i,j,k,r] = X[i,j,q] * C[k,q,r]", g["tree"][2]],
               loop_orders=["rjpqi", "rjqki", "rjki"]) == 3
    # A stored (p,q,i) and B stored (r,j,p) leave r,j,p,q,i as the only legal loop order of the first contraction
    assert chk(loop_orders=["rpqji", "rjqki", "rjki"]) == 3


def test_fusion_depth_is_the_common_loop_prefix():
    g, ext = _running_example()
    # fuse only r (X, Y become order 3): consumer of X starts r, q instead of r, j
    mo = dict(g["mode_orders"])
    red = cb.const_schedule_check(g["expression"], g["tree"], mo, ["rjpqi", "rqjki", "rjki"], ext)
    assert red == [3, 3, 0]      # Y's producer/consumer share only r as well (r,q vs r,j)
    # a loop that is not an index of the intermediate ends the fused prefix (Sec. 3.2.5, producer constraint)
    w = ttmc3_workload((6, 5, 4), 20, 8)
    red = cb.const_schedule_check(w.expression, w.tree, w.mode_orders, ["ijkb", "ijab"], w.extents)
    assert red == [1, 0]
    red = cb.const_schedule_check(w.expression, w.tree, w.mode_orders, ["ijkb", "iajb"], w.extents)
    assert red == [2, 0]         # only i is common
    red = cb.const_schedule_check(w.expression, w.tree, w.mode_orders, ["ijkb", "ajib"], w.extents)
    assert red == [3, 0]         # nothing fused: the full order-3 intermediate


@pytest.mark.parametrize("cid,family,reduced", [(1, "ttmc3", [1, 0]), (5, "network", [2, 0])])
def test_config_descriptors(cid, family, reduced):
    w = make_config(cid)
    p = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents,
                             cb.F32 if w.dtype.itemsize == 4 else cb.F64)
    assert cb.const_plan_family(p) == family
    assert [cb.const_plan_reduced_order(p, c) for c in range(len(w.tree))] == reduced
    cb.const_destroy(p)
    cb.const_destroy(p)       # idempotent


def test_other_families_and_modes():
    w = ttmc4_workload((9, 8, 7, 6), 50, 8)
    p = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    assert cb.const_plan_family(p) == "ttmc4"
    assert [cb.const_plan_reduced_order(p, c) for c in range(3)] == [1, 2, 0]      # orders 1 and 2
    w = mttkrp_workload((9, 8, 7), 50, 32)
    p = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    assert cb.const_plan_family(p) == "mttkrp3"
    # second TTMc of Sec. 5.3 (output indexed by j): same kernel family with j at the CSF root
    ext = {"i": 9, "j": 8, "k": 7, "x": 16, "z": 8}
    p = cb.const_plan_create("B[j,x,z] = T[i,j,k] * A[i,x] * C[k,z]",
                             ["S[j,i,z] = T[i,j,k] * C[k,z]", "B[j,x,z] = S[j,i,z] * A[i,x]"],
                             {"T": (1, 0, 2)}, ["jikz", "jixz"], ext, cb.F32)
    assert cb.const_plan_family(p) == "ttmc3"


def _family(**kw):
    """Family a descriptor binds to, or the status code when plan creation fails."""
    try:
        return cb.const_plan_family(cb.const_plan_create(kw["expression"], kw["tree"], kw["mode_orders"],
                                                         kw["loop_orders"], kw["extents"], kw["dtype"]))
    except cb.ConstError as e:
        return e.status


def test_legal_schedules_outside_the_families_run_on_the_generic_executor():
    w = ttmc3_workload((6, 5, 4), 20, 8)
    base = dict(expression=w.expression, tree=w.tree, mode_orders=w.mode_orders, loop_orders=w.loop_orders,
                extents=w.extents, dtype=cb.F32)
    mk = lambda **kw: _family(**dict(base, **kw))
    assert mk() == "ttmc3"
    assert mk(loop_orders=["ijkb", "iajb"]) == "tree"         # legal, but t stays order 2: no hand-written kernel
    assert mk(dtype=cb.F64) == "tree"                         # the chain kernels compute in fp32
    ext = dict(w.extents); ext["a"] = 12
    assert mk(extents=ext) == "tree"                          # rank not 8/16/32
    assert mk(expression="Y[i,b,a] = X[i,j,k] * U[j,a] * V[k,b]",
              tree=["T[i,j,b] = X[i,j,k] * V[k,b]", "Y[i,b,a] = T[i,j,b] * U[j,a]"]) == "tree"   # output layout
    big = dict(w.extents); big["i"] = 1 << 26; big["a"] = 12  # no family (rank 12), and the dense result would hold 2^31 elements or more
    assert mk(extents=big) == 2                               # beyond every executor: unsupported, not illegal
    assert mk(loop_orders=["ikjb", "ijab"]) == 3              # disagrees with CSF order (i,j,k)
    # contracting j before k is a different tree: legal only with k fused above j, which CSF (i,j,k) forbids
    assert mk(tree=["T[i,k,a] = X[i,j,k] * U[j,a]", "Y[i,a,b] = T[i,k,a] * V[k,b]"],
              loop_orders=["ikja", "ikab"]) == 3


def test_network_schedule_variants():
    w = network_workload(16, 4, 3)
    mk = lambda **kw: _family(expression=w.expression, tree=kw.get("tree", w.tree),
                              mode_orders=kw.get("mode_orders", w.mode_orders),
                              loop_orders=kw.get("loop_orders", w.loop_orders), extents=w.extents,
                              dtype=kw.get("dtype", cb.F64))
    assert mk() == "network"
    # scatter-form schedule (U stored i,j,k; W stored k,l,m): legal, generic executor
    assert mk(mode_orders={"U": (0, 1, 2), "W": (0, 1, 2)}, loop_orders=["ijkl", "iklm"]) == "tree"
    # not fused over i: T stays order 3
    assert mk(loop_orders=["ikjl", "lmik"]) == "tree"          # legal, T keeps all three modes (a global workspace)
    assert mk(loop_orders=["ikjl", "imlk"]) == 3               # W stored (l,m,k): m may not precede l
    assert mk(mode_orders={"U": (0, 2, 1), "W": (2, 1, 0)}, loop_orders=["ikjl", "imlk"]) == "tree"   # W as (m,l,k)
    assert mk(dtype=cb.F32) == "tree"


def test_malformed_descriptors():
    w = ttmc3_workload((6, 5, 4), 20, 8)
    bad = lambda **kw: _status(cb.const_plan_create, kw.get("expression", w.expression), kw.get("tree", w.tree),
                               kw.get("mode_orders", w.mode_orders), kw.get("loop_orders", w.loop_orders),
                               kw.get("extents", w.extents), cb.F32)
    assert bad(expression="Y[i,a,b] = X[i,j,k * U[j,a] * V[k,b]") == 1
    assert bad(expression="Y[i,a,b] X[i,j,k] * U[j,a] * V[k,b]") == 1
    assert bad(expression="Y[i,a,b] = X[i,j,j] * U[j,a] * V[k,b]") == 1       # repeated index in one reference
    assert bad(tree=["T[i,j,b] = X[i,j,k] * V[k,b] * U[j,a]", w.tree[1]]) == 1   # not binary
    ext = dict(w.extents); del ext["k"]
    assert bad(extents=ext) == 1
    assert bad(mode_orders={"Q": (0, 1, 2)}) == 1                              # unknown sparse tensor


def test_generic_executor_program_of_the_running_example():
    """How the compiled loop tree iterates (Sec. 4.2 structure; Fig. 5 schedule): r and j are fused and walk B, the
    other CSF operands that carry them are looked up, X and Y are 2-D workspaces cleared per (r, j), and every
    assignment keeps its own private loops in the order of its permutation."""
    g, ext = _running_example()
    p = cb.const_plan_create(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], ext, cb.F64)
    lines = [l.strip() for l in cb.const_plan_describe(p).strip().split("\n")]
    # both fused loops walk B, so the (r, j) pairs -- B's level-1 nodes -- are what the grid is spread over
    assert lines[0] == ("entry 0: blocks over r: walks B level 0; locates C level 0, D level 0"
                        " | and over j: walks B level 1; locates D level 1")
    assert lines[1].startswith("zero X(i, q) (25 elements") and lines[2].startswith("zero Y(i, k) (25 elements")
    assert lines[3].startswith("X(i, q) += A(i, p, q) * B(j, p, r)") and \
        "p: walks B level 2; locates A level 0, q: walks A level 1, i: walks A level 2" in lines[3]
    assert lines[4].startswith("Y(i, k) += X(i, q) * C(k, q, r)") and \
        "q: walks C level 1, k: walks C level 2, i: dense range 0..5" in lines[4]
    assert lines[5].startswith("R(i, j, k) += Y(i, k) * D(j, k, r)") and "k: walks D level 2, i: dense range 0..5" in lines[5]
    assert len(lines) == 6
    # a dense innermost loop is dealt to the threads together with the loop around it, unless that loop has to
    # locate an operand (p locates A, so the first assignment keeps its three loops apart)
    assert lines[4].endswith("last two dealt out as one]") and lines[5].endswith("last two dealt out as one]")
    assert lines[3].endswith("i: walks A level 2]")
    # the same holds for a TTMc at a rank the hand-written kernels do not cover: the (i, j) fibres of X are spread
    p2 = cb.const_plan_create("Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]",
                              ["T[i,j,b] = X[i,j,k] * V[k,b]", "Y[i,a,b] = T[i,j,b] * U[j,a]"],
                              {"X": (0, 1, 2)}, ["ijkb", "ijab"], {"i": 40, "j": 30, "k": 20, "a": 12, "b": 12}, cb.F64)
    assert cb.const_plan_family(p2) == "tree" and " | and over j: walks X level 1" in cb.const_plan_describe(p2)
    # unfused first contraction: X becomes a global workspace and the tree has two entries
    p = cb.const_plan_create(g["expression"], g["tree"], g["mode_orders"], ["rjpqi", "irqkj", "irjk"], ext, cb.F64)
    text = cb.const_plan_describe(p)
    assert text.count("entry ") == 2 and "zero X" not in text and "zero Y(j, k)" in text
