"""Concrete index notation of a schedule (Algorithm 1, Sec. 4.2) against what the paper prints for its
running example: the full notation of Sec. 4.1, the sequences after remove(r) and remove(j), the overall
structure, and the two-pair example that yields where(A1, forall(i, A0)).  Host only."""
import json
import os
import re

import pytest

import paper_2401_04836_b200 as cb

HERE = os.path.dirname(os.path.abspath(__file__))
EXT = {c: 4 for c in "ijkpqr"}


def squash(s):
    return re.sub(r"\s+", "", s)


@pytest.fixture(scope="module")
def golden():
    with open(os.path.join(HERE, "golden", "cin_running_example.json")) as f:
        return json.load(f)


def test_running_example_from_the_schedule_descriptor(golden):
    """The descriptor the legality checker is pinned with (references in expression order plus dp and lp)
    gives the notation printed in Sec. 4.1."""
    with open(os.path.join(HERE, "golden", "running_example_schedule.json")) as f:
        g = json.load(f)
    text = cb.const_schedule_cin(g["expression"], g["tree"], g["mode_orders"], g["loop_orders"], EXT)
    assert squash(text) == squash(golden["full"]["cin"])


@pytest.mark.parametrize("level", ["full", "after_remove_r", "after_remove_j"])
def test_each_level_of_the_recursion(golden, level):
    """The three tables of Sec. 4.2, taken as input sequences (references already in stored order)."""
    case = golden[level]
    text = cb.const_schedule_cin(golden["expression"], case["tree"], {}, case["loop_orders"], EXT, validate=False)
    assert squash(text) == squash(case["cin"])


def test_overall_structure(golden):
    text = cb.const_schedule_cin(golden["expression"], golden["full"]["tree"], {}, golden["full"]["loop_orders"], EXT,
                                 validate=False)
    shape = squash(text)
    for name, assignment in (("A0", "X(q, i) = A(p, q, i) * B(r, j, p)"), ("A1", "Y(k, i) = X(q, i) * C(r, q, k)"),
                             ("A2", "R(j, k, i) = Y(k, i) * D(r, j, k)")):
        shape = shape.replace(squash(assignment), name)
    assert shape == squash(golden["structure"])


def test_index_followed_by_an_assignment():
    """<A0,[i]>, <A1,[]>  ->  where(A1, forall(i, A0))  (Sec. 4.2)."""
    text = cb.const_schedule_cin("Z[j] = P[i,j] * Q[i] * W[j]", ["T[j] = P[i,j] * Q[i]", "Z[j] = T[j] * W[j]"], {},
                                 ["i", ""], {"i": 3, "j": 3}, validate=False)
    assert squash(text) == squash("where(Z(j) = T(j) * W(j), forall(i, T(j) = P(i, j) * Q(i)))")


def test_fused_kernel_schedules_and_errors():
    # the order-3 TTMc schedule of the benchmark: t[b] per (i, j) inside forall(i, forall(j, ...))
    text = cb.const_schedule_cin("Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]",
                                 ["T[i,j,b] = X[i,j,k] * V[k,b]", "Y[i,a,b] = T[i,j,b] * U[j,a]"],
                                 {"X": (0, 1, 2)}, ["ijkb", "ijab"], {"i": 5, "j": 4, "k": 3, "a": 2, "b": 2})
    assert squash(text) == squash("forall(i, forall(j, where(forall(a, forall(b, Y(i, a, b) = T(b) * U(j, a))), "
                                  "forall(k, forall(b, T(b) = X(i, j, k) * V(k, b))))))")
    with pytest.raises(cb.ConstError):          # a consumer that runs before its producer is not a schedule
        cb.const_schedule_cin("Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]",
                              ["Y[i,a,b] = T[i,j,b] * U[j,a]", "T[i,j,b] = X[i,j,k] * V[k,b]"],
                              {"X": (0, 1, 2)}, ["ijab", "ijkb"], {"i": 5, "j": 4, "k": 3, "a": 2, "b": 2})
