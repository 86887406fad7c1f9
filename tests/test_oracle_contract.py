"""Pins for the contraction oracle: none of these re-uses the oracle's own formula.

* dense `numpy.einsum` on densified tiny tensors (a library routine);
* closed forms (all-ones operands, identity factors, a single nonzero, rank-1 slice sums);
* the paper's three loop nests for the running example R_ijk = A_ipq B_jpr C_kqr D_jkr
  (direct n-ary Fig. 2(b), unfused Fig. 4(a), fused Fig. 4(b)) written out as Python loops;
* every contraction tree of Z_im = U_ijk V_jl W_klm (Sec. 1, Sec. 2.1 "Contraction tree");
* invariants: linearity, independence of the COO order, A >= |S|;
* planted mistakes (on the CPU, in a perturbed copy of the call) are caught by the same pins.
"""
import itertools

import numpy as np
import pytest

from oracle import contract as oc


def rand_coo(rng, dims, density, dtype=np.float64, value="normal"):
    mask = rng.random(dims) < density
    coords = [c.astype(np.int32) for c in np.nonzero(mask)]
    n = coords[0].size
    vals = rng.standard_normal(n) if value == "normal" else np.ones(n)
    perm = rng.permutation(n)
    return [c[perm] for c in coords], vals[perm].astype(dtype)


def densify(coords, vals, dims):
    D = np.zeros(dims, dtype=np.float64)
    D[tuple(coords)] = vals
    return D


@pytest.mark.parametrize("density", [0.05, 0.4, 1.0])
@pytest.mark.parametrize("dims,ra,rb", [((5, 4, 6), 3, 2), ((2, 7, 3), 4, 4)])
def test_ttmc3_vs_einsum(dims, ra, rb, density):
    rng = np.random.default_rng(1)
    coords, vals = rand_coo(rng, dims, density)
    U, V = rng.standard_normal((dims[1], ra)), rng.standard_normal((dims[2], rb))
    S, A = oc.ttmc3(coords, vals, U, V, dims[0])
    X = densify(coords, vals, dims)
    np.testing.assert_allclose(S, np.einsum("ijk,ja,kb->iab", X, U, V), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,ja,kb->iab", abs(X), abs(U), abs(V)), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("density", [0.1, 1.0])
def test_ttmc4_vs_einsum(density):
    rng = np.random.default_rng(2)
    dims = (4, 3, 5, 2)
    coords, vals = rand_coo(rng, dims, density)
    U, V, W = (rng.standard_normal((dims[1], 2)), rng.standard_normal((dims[2], 3)),
               rng.standard_normal((dims[3], 4)))
    S, A = oc.ttmc4(coords, vals, U, V, W, dims[0])
    X = densify(coords, vals, dims)
    np.testing.assert_allclose(S, np.einsum("ijkl,ja,kb,lc->iabc", X, U, V, W), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijkl,ja,kb,lc->iabc", abs(X), abs(U), abs(V), abs(W)),
                               rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("density", [0.1, 1.0])
def test_mttkrp_vs_einsum(density):
    rng = np.random.default_rng(3)
    dims = (6, 5, 4)
    coords, vals = rand_coo(rng, dims, density)
    B, C = rng.standard_normal((dims[1], 3)), rng.standard_normal((dims[2], 3))
    S, A = oc.mttkrp3(coords, vals, B, C, dims[0])
    X = densify(coords, vals, dims)
    np.testing.assert_allclose(S, np.einsum("ijk,jr,kr->ir", X, B, C), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,jr,kr->ir", abs(X), abs(B), abs(C)), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("density", [0.15, 1.0])
def test_network_vs_einsum_and_all_trees(density):
    """Z_im = sum_jkl U_ijk V_jl W_klm; every binarisation of the network gives the same result."""
    rng = np.random.default_rng(4)
    ni, nj, nk, nl, nm = 5, 4, 3, 6, 7
    uc, uv = rand_coo(rng, (ni, nj, nk), density)
    wc, wv = rand_coo(rng, (nk, nl, nm), density)
    V = rng.standard_normal((nj, nl))
    S, A = oc.network(uc, uv, V, wc, wv, ni, nk, nm)
    U, W = densify(uc, uv, (ni, nj, nk)), densify(wc, wv, (nk, nl, nm))
    ref = np.einsum("ijk,jl,klm->im", U, V, W)
    np.testing.assert_allclose(S, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,jl,klm->im", abs(U), abs(V), abs(W)), rtol=1e-12, atol=1e-13)
    t1 = np.einsum("ikl,klm->im", np.einsum("ijk,jl->ikl", U, V), W)        # (U V) W
    t2 = np.einsum("ijk,jkm->im", U, np.einsum("jl,klm->jkm", V, W))        # U (V W)
    t3 = np.einsum("ijlm,jl->im", np.einsum("ijk,klm->ijlm", U, W), V)      # (U W) V
    for t in (t1, t2, t3):
        np.testing.assert_allclose(S, t, rtol=1e-11, atol=1e-12)


def test_generic_matches_specialised_and_einsum():
    rng = np.random.default_rng(5)
    dims = (3, 4, 3)
    coords, vals = rand_coo(rng, dims, 0.4)
    U, V = rng.standard_normal((4, 2)), rng.standard_normal((3, 3))
    ext = {"i": 3, "j": 4, "k": 3, "a": 2, "b": 3}
    Sg, Ag = oc.nary_direct("Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]", {"X": (coords, vals), "U": U, "V": V}, ext)
    Sc, Ac = oc.ttmc3(coords, vals, U, V, 3)
    np.testing.assert_allclose(Sg, Sc, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(Ag, Ac, rtol=1e-12, atol=1e-13)
    B, C = rng.standard_normal((4, 2)), rng.standard_normal((3, 2))
    Sg, _ = oc.nary_direct("A[i,r] = X[i,j,k] * B[j,r] * C[k,r]", {"X": (coords, vals), "B": B, "C": C},
                           {"i": 3, "j": 4, "k": 3, "r": 2})
    np.testing.assert_allclose(Sg, oc.mttkrp3(coords, vals, B, C, 3)[0], rtol=1e-12, atol=1e-13)


def _running_example(rng, n, density):
    """Four sparse order-3 inputs of the running example, all extents n."""
    return {name: rand_coo(rng, (n, n, n), density) for name in "ABCD"}


def test_running_example_three_loop_nests():
    """Fig. 2(b) direct nest, Fig. 4(a) unfused sequence and Fig. 4(b) fused nest all agree with the oracle."""
    rng = np.random.default_rng(6)
    n = 3
    ops = _running_example(rng, n, 0.5)
    expr = "R[i,j,k] = A[i,p,q] * B[j,p,r] * C[k,q,r] * D[j,k,r]"
    S, A_abs = oc.nary_direct(expr, ops, {x: n for x in "ijkpqr"})
    A, B, C, D = (densify(*ops[x], (n, n, n)) for x in "ABCD")
    rg = range(n)
    # Fig. 2(b): one loop per index, one statement
    R_direct = np.zeros((n, n, n))
    for i, j, k, p, q, r in itertools.product(rg, repeat=6):
        R_direct[i, j, k] += A[i, p, q] * B[j, p, r] * C[k, q, r] * D[j, k, r]
    # Fig. 4(a): three perfect nests with full-order intermediates
    X = np.zeros((n,) * 4); Y = np.zeros((n,) * 4); R_unfused = np.zeros((n,) * 3)
    for i, j, p, q, r in itertools.product(rg, repeat=5):
        X[i, j, q, r] += A[i, p, q] * B[j, p, r]
    for i, j, k, q, r in itertools.product(rg, repeat=5):
        Y[i, j, k, r] += X[i, j, q, r] * C[k, q, r]
    for i, j, k, r in itertools.product(rg, repeat=4):
        R_unfused[i, j, k] += Y[i, j, k, r] * D[j, k, r]
    # Fig. 4(b): loops i, j fused; X and Y shrink to 2-D and are reset per (i, j)
    R_fused = np.zeros((n,) * 3)
    for i, j in itertools.product(rg, repeat=2):
        Xs = np.zeros((n, n)); Ys = np.zeros((n, n))
        for p, q, r in itertools.product(rg, repeat=3):
            Xs[q, r] += A[i, p, q] * B[j, p, r]
        for k, q, r in itertools.product(rg, repeat=3):
            Ys[k, r] += Xs[q, r] * C[k, q, r]
        for k, r in itertools.product(rg, repeat=2):
            R_fused[i, j, k] += Ys[k, r] * D[j, k, r]
    for R in (R_direct, R_unfused, R_fused):
        np.testing.assert_allclose(S, R, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(S, np.einsum("ipq,jpr,kqr,jkr->ijk", A, B, C, D), rtol=1e-11, atol=1e-12)
    assert np.all(A_abs >= np.abs(S) - 1e-12)


def test_closed_form_all_ones():
    """All-ones dense operands: every output counts the contributing index combinations."""
    dims = (3, 4, 5)
    coords = [c.ravel().astype(np.int32) for c in np.indices(dims)]
    vals = np.ones(coords[0].size)
    S, A = oc.ttmc3(coords, vals, np.ones((4, 2)), np.ones((5, 3)), 3)
    assert np.all(S == 4 * 5) and np.all(A == 4 * 5)
    S, _ = oc.mttkrp3(coords, vals, np.ones((4, 2)), np.ones((5, 2)), 3)
    assert np.all(S == 20)
    d4 = (2, 3, 2, 4)
    c4 = [c.ravel().astype(np.int32) for c in np.indices(d4)]
    S, _ = oc.ttmc4(c4, np.ones(c4[0].size), np.ones((3, 2)), np.ones((2, 2)), np.ones((4, 3)), 2)
    assert np.all(S == 3 * 2 * 4)
    # network: Z[i,m] = Nj * Nk * Nl when everything is one
    uc = [c.ravel().astype(np.int32) for c in np.indices((2, 3, 4))]
    wc = [c.ravel().astype(np.int32) for c in np.indices((4, 5, 6))]
    S, _ = oc.network(uc, np.ones(24), np.ones((3, 5)), wc, np.ones(120), 2, 4, 6)
    assert np.all(S == 3 * 4 * 5)


def test_closed_form_identity_factors_and_single_nonzero():
    rng = np.random.default_rng(7)
    dims = (4, 3, 5)
    coords, vals = rand_coo(rng, dims, 0.5)
    # identity factors return the densified tensor itself
    S, _ = oc.ttmc3(coords, vals, np.eye(3), np.eye(5), 4)
    np.testing.assert_array_equal(S, densify(coords, vals, dims))
    # MTTKRP with identity factors picks the entries with j = k = r
    n = 4
    c2, v2 = rand_coo(rng, (3, n, n), 0.7)
    S, _ = oc.mttkrp3(c2, v2, np.eye(n), np.eye(n), 3)
    X = densify(c2, v2, (3, n, n))
    np.testing.assert_array_equal(S, np.stack([np.diag(X[i]) for i in range(3)]))
    # a single nonzero gives one scaled outer product in one slice
    U, V = rng.standard_normal((3, 2)), rng.standard_normal((5, 3))
    S, A = oc.ttmc3([np.array([2]), np.array([1]), np.array([4])], np.array([-1.5]), U, V, 4)
    expect = np.zeros((4, 2, 3)); expect[2] = -1.5 * np.outer(U[1], V[4])
    np.testing.assert_allclose(S, expect, rtol=1e-15)
    np.testing.assert_allclose(A, np.abs(expect), rtol=1e-15)
    # rank-1 all-ones factors: slice sums of X
    S, _ = oc.ttmc3(coords, vals, np.ones((3, 1)), np.ones((5, 1)), 4)
    np.testing.assert_allclose(S[:, 0, 0], densify(coords, vals, dims).sum(axis=(1, 2)), rtol=1e-13)


def test_invariants_linearity_and_order():
    rng = np.random.default_rng(8)
    dims = (6, 5, 4)
    coords, vals = rand_coo(rng, dims, 0.3)
    U, V = rng.standard_normal((5, 3)), rng.standard_normal((4, 2))
    S, A = oc.ttmc3(coords, vals, U, V, 6)
    perm = rng.permutation(vals.size)
    S2, A2 = oc.ttmc3([c[perm] for c in coords], vals[perm], U, V, 6)
    np.testing.assert_allclose(S, S2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(A, A2, rtol=1e-12, atol=1e-14)
    S3, _ = oc.ttmc3(coords, 2.5 * vals, U, V, 6)
    np.testing.assert_allclose(S3, 2.5 * S, rtol=1e-13)
    U2 = rng.standard_normal(U.shape)
    Sa, _ = oc.ttmc3(coords, vals, U + U2, V, 6)
    Sb, _ = oc.ttmc3(coords, vals, U2, V, 6)
    np.testing.assert_allclose(Sa, S + Sb, rtol=1e-10, atol=1e-12)
    assert np.all(A >= np.abs(S))
    # rows that hold no nonzero stay exactly zero
    empty_rows = np.setdiff1d(np.arange(6), coords[0])
    assert np.all(S[empty_rows] == 0)


def test_float32_inputs_are_widened_exactly():
    rng = np.random.default_rng(9)
    dims = (4, 4, 4)
    coords, vals = rand_coo(rng, dims, 0.5, dtype=np.float32)
    U = rng.standard_normal((4, 2)).astype(np.float32)
    V = rng.standard_normal((4, 2)).astype(np.float32)
    S, _ = oc.ttmc3(coords, vals, U, V, 4)
    ref = np.einsum("ijk,ja,kb->iab", densify(coords, vals.astype(np.float64), dims),
                    U.astype(np.float64), V.astype(np.float64))
    np.testing.assert_allclose(S, ref, rtol=1e-13, atol=1e-14)


def test_compensated_network_sum_beats_tolerance():
    """The fp64 network tolerance is 1e-12 * A; the oracle's own error must be far below it.
    Check against exact rational arithmetic on integer-valued inputs scaled by powers of two."""
    rng = np.random.default_rng(10)
    ni, nj, nk, nl, nm = 2, 6, 5, 6, 3
    uc, _ = rand_coo(rng, (ni, nj, nk), 0.9)
    wc, _ = rand_coo(rng, (nk, nl, nm), 0.9)
    uv = rng.integers(-2**20, 2**20, uc[0].size).astype(np.float64)
    wv = rng.integers(-2**20, 2**20, wc[0].size).astype(np.float64)
    V = rng.integers(-2**12, 2**12, (nj, nl)).astype(np.float64)
    S, A = oc.network(uc, uv, V, wc, wv, ni, nk, nm)
    exact = np.zeros((ni, nm), dtype=object)
    for e in range(uv.size):
        for f in range(wv.size):
            if uc[2][e] == wc[0][f]:
                exact[uc[0][e], wc[2][f]] += int(uv[e]) * int(V[uc[1][e], wc[1][f]]) * int(wv[f])
    err = np.abs(S - exact.astype(np.float64))
    assert np.all(err <= 1e-15 * A + 1e-300)


def test_planted_mistakes_are_caught():
    """Plausible slips (swapped factors, transposed factor, dropped abs) change the result visibly."""
    rng = np.random.default_rng(11)
    dims = (4, 5, 5)
    coords, vals = rand_coo(rng, dims, 0.4)
    U, V = rng.standard_normal((5, 3)), rng.standard_normal((5, 3))
    ref = np.einsum("ijk,ja,kb->iab", densify(coords, vals, dims), U, V)
    S_swapped, _ = oc.ttmc3(coords, vals, V, U, 4)                        # factors exchanged
    assert not np.allclose(S_swapped, ref, rtol=1e-6)
    S_modes, _ = oc.ttmc3([coords[0], coords[2], coords[1]], vals, U, V, 4)   # j and k exchanged
    assert not np.allclose(S_modes, ref, rtol=1e-6)
    S_ok, A_ok = oc.ttmc3(coords, vals, U, V, 4)
    assert np.allclose(S_ok, ref, rtol=1e-12)
    assert not np.allclose(A_ok, np.abs(S_ok))                            # A is not |S|


def test_rejects_out_of_range_coordinates():
    with pytest.raises(ValueError):
        oc.ttmc3([np.array([0]), np.array([9]), np.array([0])], np.array([1.0]), np.ones((3, 2)), np.ones((3, 2)), 2)
    with pytest.raises(ValueError):
        oc.ttmc3([np.array([5]), np.array([0]), np.array([0])], np.array([1.0]), np.ones((3, 2)), np.ones((3, 2)), 2)


def test_einsum_evaluator_agrees_with_the_loop_nest_evaluator():
    """`nary_einsum` (densify + numpy.einsum) against `nary_direct` (Python loops over stored nonzeros) on the
    running example, an order-4 MTTKRP and a network times a sparse 0/1 map; and a closed form: with every stored
    value 1 and dense factors of ones, an output element counts the index combinations that reach it."""
    rng = np.random.default_rng(16)
    n = 3
    ops = _running_example(rng, n, 0.6)
    expr = "R[i,j,k] = A[i,p,q] * B[j,p,r] * C[k,q,r] * D[j,k,r]"
    ext = {x: n for x in "ijkpqr"}
    S1, A1 = oc.nary_direct(expr, ops, ext)
    S2, A2 = oc.nary_einsum(expr, ops, ext)
    np.testing.assert_allclose(S2, S1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A2, A1, rtol=1e-12, atol=1e-13)
    assert np.all(A2 >= np.abs(S2) - 1e-12) and np.any(A2 > np.abs(S2) + 1e-9)      # signs do cancel somewhere

    dims = (4, 3, 2, 3)
    X = rand_coo(rng, dims, 0.3)
    fac = {"B": rng.standard_normal((3, 2)), "C": rng.standard_normal((2, 2)), "D": rng.standard_normal((3, 2))}
    expr4 = "M[i,r] = X[i,j,k,l] * B[j,r] * C[k,r] * D[l,r]"
    ext4 = {"i": 4, "j": 3, "k": 2, "l": 3, "r": 2}
    S1, A1 = oc.nary_direct(expr4, dict(fac, X=X), ext4)
    S2, A2 = oc.nary_einsum(expr4, dict(fac, X=X), ext4)
    np.testing.assert_allclose(S2, S1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A2, A1, rtol=1e-12, atol=1e-13)

    I3 = rand_coo(rng, (3, 4, 3), 0.5)
    L = rand_coo(rng, (3, 2), 0.5)
    L = (L[0], np.ones_like(L[1]))
    Cm, Pm = rng.standard_normal((4, 2)), rng.standard_normal((3, 4))
    exprm = "E[k,i,m] = I[k,u,v] * C[u,i] * P[v,m] * L[k,i]"
    extm = {"k": 3, "u": 4, "v": 3, "i": 2, "m": 4}
    S1, A1 = oc.nary_direct(exprm, {"I": I3, "C": Cm, "P": Pm, "L": L}, extm)
    S2, A2 = oc.nary_einsum(exprm, {"I": I3, "C": Cm, "P": Pm, "L": L}, extm)
    np.testing.assert_allclose(S2, S1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(A2, A1, rtol=1e-12, atol=1e-13)
    mask = densify(*L, (3, 2))
    assert np.all(S2[mask == 0] == 0)                                   # nothing outside the map

    ones = {"X": (X[0], np.ones_like(X[1])), "B": np.ones((3, 2)), "C": np.ones((2, 2)), "D": np.ones((3, 2))}
    S, A = oc.nary_einsum(expr4, ones, ext4)
    per_slice = np.bincount(X[0][0], minlength=4)
    np.testing.assert_array_equal(S, np.repeat(per_slice[:, None], 2, axis=1))
    np.testing.assert_array_equal(A, S)
