"""GPU CSF builder vs the CSF oracle: bit-exact arrays for every mode order, edge cases, error codes."""
import itertools

import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from workloads import generators as gen
from workloads import make_config
from tests.gpu_util import assert_csf_equal, build_csf, csf_to_host, to_dev

pytestmark = pytest.mark.gpu


def random_op(rng, dims, nnz, dtype=np.float32):
    op = gen._uniform_tensor(dims, nnz, rng, "pm1", dtype)
    return op


@pytest.mark.parametrize("dims,nnz", [((7, 5), 20), ((6, 5, 9), 120), ((5, 4, 3, 6), 200), ((37, 41, 29), 9000)])
def test_every_mode_order_small(dims, nnz):
    rng = np.random.default_rng(len(dims) * 1000 + nnz)
    op = random_op(rng, dims, nnz)
    for mo in itertools.permutations(range(len(dims))):
        h = build_csf(op, mo)
        assert_csf_equal(h, op, mo)
        cb.const_destroy(h)


@pytest.mark.parametrize("nnz", [4096, 4097, 3 * 4096 + 17, 250_003])
def test_several_tiles_and_ragged_tail(nnz):
    rng = np.random.default_rng(nnz)
    op = random_op(rng, (300, 1000, 777), nnz)
    for mo in [(0, 1, 2), (2, 0, 1)]:
        h = build_csf(op, mo)
        assert_csf_equal(h, op, mo)


@pytest.mark.parametrize("dims,nnz", [((512, 512, 512), 250_003),      # 27 key bits: three 9-bit digits
                                      ((512, 256), 100_000),           # 17 bits: one 9-bit and one 8-bit digit
                                      ((2048, 2048, 2048, 512), 70_001),   # 42 bits: 9 9 8 8 8
                                      ((3, 2, 2), 12)])                # 5 bits: one short digit
def test_digit_widths(dims, nnz):
    rng = np.random.default_rng(sum(dims) + nnz)
    for dtype in (np.float32, np.float64):
        op = random_op(rng, dims, nnz, dtype=dtype)
        mo = tuple(reversed(range(len(dims))))
        assert_csf_equal(build_csf(op, mo), op, mo)


def test_order4_wide_key_and_fp64_values():
    rng = np.random.default_rng(5)
    op = random_op(rng, (20000, 20000, 20000, 20000), 60_000)        # 60-bit key, 8 passes
    h = build_csf(op, (0, 1, 2, 3))
    assert_csf_equal(h, op, (0, 1, 2, 3))
    op64 = random_op(rng, (1024, 1024, 128), 50_000, dtype=np.float64)
    for mo in [(0, 2, 1), (2, 1, 0)]:
        assert_csf_equal(build_csf(op64, mo), op64, mo)


def test_skewed_slices_like_the_benchmark():
    w = make_config(2, scale=0.004)                                   # ~300k nonzeros, Zipf slices and coordinates
    op = w.sparse["X"]
    h = build_csf(op, (0, 1, 2))
    assert_csf_equal(h, op, (0, 1, 2))
    counts = cb.const_csf_bin_counts(h)
    assert counts["light"] + counts["heavy"] + counts["giant"] == 12_000


def test_edge_cases():
    S = gen.SparseOperand
    i32 = lambda *a: np.array(a, dtype=np.int32)
    # empty tensor
    op = S([i32(), i32(), i32()], np.zeros(0, np.float32), (4, 5, 6))
    h = build_csf(op, (0, 1, 2))
    assert_csf_equal(h, op, (0, 1, 2))
    assert cb.const_csf_bin_counts(h)["items"] == 0
    # one nonzero at the largest coordinates; -0.0 keeps its sign bit; extents that are not powers of two
    op = S([i32(4), i32(2), i32(6)], np.array([-0.0], np.float32), (5, 3, 7))
    for mo in [(0, 1, 2), (2, 0, 1)]:
        assert_csf_equal(build_csf(op, mo), op, mo)
    # stored zeros stay; a single giant slice; empty slices do not appear
    n = 20_000
    rng = np.random.default_rng(1)
    j = rng.permutation(200 * 300)[:n]
    op = S([np.full(n, 3, np.int32), (j // 300).astype(np.int32), (j % 300).astype(np.int32)],
           np.where(rng.random(n) < 0.1, 0.0, rng.standard_normal(n)).astype(np.float32), (9, 200, 300))
    h = build_csf(op, (0, 1, 2))
    assert_csf_equal(h, op, (0, 1, 2))
    pos, crd, _ = csf_to_host(h)
    assert crd[0].tolist() == [3]
    # extent 1 modes and the maximum extent of a mode
    op = S([i32(0, 0), i32(0, 2**31 - 2), i32(1, 0)], np.array([1, 2], np.float32), (1, 2**31 - 1, 2))
    assert_csf_equal(build_csf(op, (1, 0, 2)), op, (1, 0, 2))


def test_error_codes():
    S = gen.SparseOperand
    i32 = lambda *a: np.array(a, dtype=np.int32)
    dup = S([i32(1, 2, 1), i32(0, 1, 0), i32(3, 3, 3)], np.ones(3, np.float32), (4, 4, 4))
    with pytest.raises(cb.ConstError) as e:
        build_csf(dup, (0, 1, 2))
    assert e.value.status == 4
    for bad in (S([i32(4), i32(0), i32(0)], np.ones(1, np.float32), (4, 4, 4)),
                S([i32(0), i32(-1), i32(0)], np.ones(1, np.float32), (4, 4, 4))):
        with pytest.raises(cb.ConstError) as e:
            build_csf(bad, (0, 1, 2))
        assert e.value.status == 5
    # the context stays usable after an error
    ok = S([i32(1), i32(1), i32(1)], np.ones(1, np.float32), (4, 4, 4))
    assert_csf_equal(build_csf(ok, (0, 1, 2)), ok, (0, 1, 2))
    with pytest.raises(cb.ConstError) as e:
        cb.const_csf_build([to_dev(i32(0))] * 3, to_dev(np.ones(1, np.float32)), (4, 4, 4), (0, 0, 1))
    assert e.value.status == 1
    with pytest.raises(cb.ConstError) as e:                         # key wider than 64 bits
        cb.const_csf_build([to_dev(i32(0))] * 4, to_dev(np.ones(1, np.float32)), (2**31 - 1,) * 4, (0, 1, 2, 3))
    assert e.value.status == 2
