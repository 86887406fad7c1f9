"""Oracle front end for whole workloads.  TEST INFRASTRUCTURE ONLY (see package docstring).

Picks the oracle routine that evaluates a workload's expression (Sec. 2.1 definition, see
`contract.py`) and hands it the workload's COO arrays and dense factors.  No arithmetic of its own.
"""
from __future__ import annotations

import numpy as np

from . import contract as oc


def _rows_of(op, rows, mode=0):
    """The nonzeros of a COO operand whose coordinate along `mode` lies in `rows` (pure filtering)."""
    sel = np.isin(op.coords[mode], np.asarray(rows))
    return [np.ascontiguousarray(c[sel]) for c in op.coords], np.ascontiguousarray(op.vals[sel])


def evaluate(w, rows=None):
    """(S, A) of the workload's expression, both shaped like its output.

    rows = only the nonzeros whose output row (first index of the result) lies in `rows` take
    part; the other rows of S and A come back as zeros.  The result rows that are evaluated are
    exact for the full tensor, because an output row depends on the nonzeros of its slice only.
    """
    fam = w.family
    if fam == "network":
        U, W = w.sparse["U"], w.sparse["W"]
        uc, uv = (U.coords, U.vals) if rows is None else _rows_of(U, rows)
        return oc.network(uc, uv, w.dense["V"], W.coords, W.vals, w.extents["i"], w.extents["k"], w.extents["m"])
    X = w.sparse["X"]
    xc, xv = (X.coords, X.vals) if rows is None else _rows_of(X, rows)
    if fam == "ttmc3":
        return oc.ttmc3(xc, xv, w.dense["U"], w.dense["V"], X.dims[0])
    if fam == "ttmc4":
        return oc.ttmc4(xc, xv, w.dense["U"], w.dense["V"], w.dense["W"], X.dims[0])
    if fam == "mttkrp":
        return oc.mttkrp3(xc, xv, w.dense["B"], w.dense["C"], X.dims[0])
    raise ValueError(fam)
