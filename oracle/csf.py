"""CSF oracle.  TEST INFRASTRUCTURE ONLY (see package docstring).

Compressed Sparse Fiber (paper Sec. 2.1, "CSF representation"): a sparse tensor is stored as a
tree fixed by a permutation of its modes.  Level l of the tree holds one node for every distinct
prefix (c_0, ..., c_l) of the permuted coordinate tuples; the node stores c_l; the leaves carry
the values; an auxiliary root ties the level-0 nodes together.

Concrete arrays (the paper leaves the encoding open; this is the usual one):
  * nodes of each level are listed in lexicographic order of their prefixes;
  * crd[l][n]  = coordinate stored by node n of level l;
  * pos[l][p]  = index, in level l, of the first child of node p of level l-1, with
                 pos[l][n_{l-1}] = n_l closing the last segment; pos[0] = [0, n_0] (children of the root);
  * vals[n]    = value of leaf n (leaves are the nodes of the last level).
All levels are compressed: a coordinate that has no nonzero below it has no node.  Stored zeros
are kept.  Repeated coordinate tuples are an error, because nz(T) is a set.

`build` is the definition written with a library sort; `build_bruteforce` builds the same tree
as nested dictionaries, one insertion per nonzero, for pinning on tiny inputs.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np


class DuplicateCoordinate(ValueError):
    pass


def build(coords: Sequence[np.ndarray], vals: np.ndarray, mode_order: Sequence[int]):
    """Return (pos, crd, vals_sorted): lists with one int32 array per level, and the leaf values."""
    order = len(mode_order)
    if sorted(mode_order) != list(range(order)) or len(coords) != order:
        raise ValueError("mode_order must be a permutation of the modes")
    nnz = int(np.asarray(vals).shape[0])
    lev = [np.asarray(coords[m]) for m in mode_order]           # lev[l] = coordinates stored at level l
    if nnz == 0:
        pos = [np.zeros(2 if l == 0 else 1, dtype=np.int32) for l in range(order)]
        return pos, [np.zeros(0, dtype=np.int32) for _ in range(order)], np.asarray(vals).copy()
    perm = np.lexsort(tuple(lev[::-1]))                          # primary key = level 0
    lev = [c[perm] for c in lev]
    v = np.asarray(vals)[perm]
    # new_node[l][e] is True when element e starts a new prefix of length l+1
    differs = np.zeros(nnz, dtype=bool)
    differs[0] = True
    new_node = []
    for l in range(order):
        differs = differs.copy()
        differs[1:] |= lev[l][1:] != lev[l][:-1]
        new_node.append(differs)
    if not new_node[-1].all():
        raise DuplicateCoordinate("the same coordinate tuple appears more than once")
    crd = [lev[l][new_node[l]].astype(np.int32) for l in range(order)]
    n = [int(c.shape[0]) for c in crd]
    node_id = [np.cumsum(new_node[l]) - 1 for l in range(order)]  # node of level l that element e lies under
    pos = [np.array([0, n[0]], dtype=np.int32)]
    for l in range(1, order):
        first_child = node_id[l][new_node[l - 1]]                 # one entry per node of level l-1
        pos.append(np.concatenate([first_child, [n[l]]]).astype(np.int32))
    return pos, crd, v.copy()


def build_bruteforce(coords: Sequence[np.ndarray], vals: np.ndarray, mode_order: Sequence[int]):
    """Same arrays, from a tree of nested dicts filled one nonzero at a time (tiny inputs)."""
    order = len(mode_order)
    root: Dict = {}
    for e in range(len(vals)):
        node = root
        for l in range(order):
            c = int(coords[mode_order[l]][e])
            if l == order - 1:
                if c in node:
                    raise DuplicateCoordinate("the same coordinate tuple appears more than once")
                node[c] = vals[e]
            else:
                node = node.setdefault(c, {})
    crd: List[List[int]] = [[] for _ in range(order)]
    pos: List[List[int]] = [[0] for _ in range(order)]
    leaves = []

    def walk(node: Dict, l: int):
        for c in sorted(node):
            crd[l].append(c)
            if l == order - 1:
                leaves.append(node[c])
            else:
                walk(node[c], l + 1)
                pos[l + 1].append(len(crd[l + 1]))
    walk(root, 0)
    pos[0].append(len(crd[0]))
    return ([np.array(p, dtype=np.int32) for p in pos], [np.array(c, dtype=np.int32) for c in crd],
            np.array(leaves, dtype=np.asarray(vals).dtype))


def expand(pos, crd, vals, mode_order: Sequence[int]):
    """Inverse of `build`: walk the tree and return COO coordinates (in mode numbering) and values."""
    order = len(mode_order)
    nnz = len(vals)
    per_level = [None] * order
    idx = np.arange(nnz)
    per_level[order - 1] = np.asarray(crd[order - 1])[idx]
    for l in range(order - 1, 0, -1):
        parent = np.searchsorted(np.asarray(pos[l]), idx, side="right") - 1   # node of level l-1 owning child idx
        per_level[l - 1] = np.asarray(crd[l - 1])[parent]
        idx = parent
    coords = [None] * order
    for l, m in enumerate(mode_order):
        coords[m] = per_level[l].astype(np.int32)
    return coords, np.asarray(vals)
