"""Pins for the CSF oracle (Sec. 2.1, CSF representation).

* a hand-expanded order-4 example (tests/golden/csf_order4_example.json);
* a brute-force tree of nested dicts, for every mode permutation of random tiny tensors;
* order 2 reduces to textbook (doubly) compressed sparse rows: cross-checked with scipy;
* structural invariants and the round trip CSF -> COO -> same sorted set.
"""
import itertools
import json
import os

import numpy as np
import pytest
import scipy.sparse as sp

from oracle import csf as ocsf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_coo(rng, dims, density):
    mask = rng.random(dims) < density
    coords = [c.astype(np.int32) for c in np.nonzero(mask)]
    n = coords[0].size
    perm = rng.permutation(n)
    return [c[perm] for c in coords], rng.standard_normal(n).astype(np.float32)[perm]


def test_hand_worked_order4_example():
    with open(os.path.join(GOLDEN, "csf_order4_example.json")) as f:
        g = json.load(f)
    coords = [np.array(c, dtype=np.int32) for c in g["coords"]]
    vals = np.array(g["vals"], dtype=np.float32)
    rng = np.random.default_rng(0)
    perm = rng.permutation(vals.size)                      # COO order must not matter
    for case in g["cases"]:
        pos, crd, v = ocsf.build([c[perm] for c in coords], vals[perm], case["mode_order"])
        for l in range(4):
            assert crd[l].tolist() == case["crd"][l], (case["mode_order"], l)
            assert pos[l].tolist() == case["pos"][l], (case["mode_order"], l)
        assert v.tolist() == case["vals"]


@pytest.mark.parametrize("dims", [(4, 3, 5), (3, 3, 2, 4), (6, 7)])
@pytest.mark.parametrize("density", [0.1, 0.6, 1.0])
def test_matches_bruteforce_for_every_mode_order(dims, density):
    rng = np.random.default_rng(hash((dims, density)) % 2**32)
    coords, vals = rand_coo(rng, dims, density)
    for mo in itertools.permutations(range(len(dims))):
        pos, crd, v = ocsf.build(coords, vals, mo)
        bpos, bcrd, bv = ocsf.build_bruteforce(coords, vals, mo)
        for l in range(len(dims)):
            np.testing.assert_array_equal(pos[l], bpos[l])
            np.testing.assert_array_equal(crd[l], bcrd[l])
        assert v.tobytes() == bv.tobytes()


def test_order2_is_doubly_compressed_csr():
    rng = np.random.default_rng(3)
    dims = (9, 7)
    coords, vals = rand_coo(rng, dims, 0.3)
    pos, crd, v = ocsf.build(coords, vals, (0, 1))
    M = sp.coo_matrix((vals.astype(np.float64), (coords[0], coords[1])), shape=dims).tocsr()
    M.sort_indices()
    nonempty = np.nonzero(np.diff(M.indptr))[0]
    np.testing.assert_array_equal(crd[0], nonempty)
    np.testing.assert_array_equal(pos[1], np.concatenate([M.indptr[nonempty], [M.nnz]]))
    np.testing.assert_array_equal(crd[1], M.indices)
    np.testing.assert_array_equal(v.astype(np.float64), M.data)
    # the transposed mode order is CSC
    pos, crd, v = ocsf.build(coords, vals, (1, 0))
    Mc = M.tocsc(); Mc.sort_indices()
    nonempty = np.nonzero(np.diff(Mc.indptr))[0]
    np.testing.assert_array_equal(crd[0], nonempty)
    np.testing.assert_array_equal(crd[1], Mc.indices)
    np.testing.assert_array_equal(v.astype(np.float64), Mc.data)


def test_invariants_and_round_trip():
    rng = np.random.default_rng(4)
    dims = (7, 5, 6, 3)
    coords, vals = rand_coo(rng, dims, 0.08)
    for mo in [(0, 1, 2, 3), (2, 0, 3, 1), (3, 2, 1, 0)]:
        pos, crd, v = ocsf.build(coords, vals, mo)
        n = [len(c) for c in crd]
        assert n[-1] == vals.size
        assert pos[0].tolist() == [0, n[0]]
        for l in range(1, 4):
            assert pos[l][0] == 0 and pos[l][-1] == n[l] and len(pos[l]) == n[l - 1] + 1
            assert np.all(np.diff(pos[l]) >= 1)              # every stored node has a child
        for l in range(4):
            for p in range(len(pos[l]) - 1):
                seg = crd[l][pos[l][p]:pos[l][p + 1]]
                assert np.all(np.diff(seg) > 0)              # strictly increasing inside a parent
        back, bv = ocsf.expand(pos, crd, v, mo)
        key = lambda cs: np.lexsort(tuple(cs[::-1]))
        a, b = key(coords), key(back)
        for m in range(4):
            np.testing.assert_array_equal(coords[m][a], back[m][b])
        assert vals[a].tobytes() == bv[b].tobytes()


def test_edge_cases():
    # empty tensor
    pos, crd, v = ocsf.build([np.zeros(0, np.int32)] * 3, np.zeros(0, np.float32), (0, 1, 2))
    assert pos[0].tolist() == [0, 0] and all(len(c) == 0 for c in crd) and len(v) == 0
    # one nonzero, at the largest coordinate
    pos, crd, v = ocsf.build([np.array([4]), np.array([2]), np.array([6])], np.array([-0.0], np.float32), (2, 0, 1))
    assert [c.tolist() for c in crd] == [[6], [4], [2]]
    assert [p.tolist() for p in pos] == [[0, 1], [0, 1], [0, 1]]
    assert np.signbit(v[0])                                   # value bits move untouched
    # stored zeros stay
    pos, crd, v = ocsf.build([np.array([0, 0])] * 1 + [np.array([0, 1])], np.array([0.0, 1.0], np.float32), (0, 1))
    assert crd[1].tolist() == [0, 1] and v.tolist() == [0.0, 1.0]
    # duplicates are an error
    with pytest.raises(ocsf.DuplicateCoordinate):
        ocsf.build([np.array([1, 1]), np.array([2, 2])], np.array([1.0, 2.0], np.float32), (0, 1))
    with pytest.raises(ocsf.DuplicateCoordinate):
        ocsf.build_bruteforce([np.array([1, 1]), np.array([2, 2])], np.array([1.0, 2.0], np.float32), (0, 1))
