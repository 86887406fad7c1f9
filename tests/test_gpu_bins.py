"""The load balancer's work lists, checked directly (not only through the outputs they lead to).

For every threshold setting: each root slice appears in exactly one place -- the light list, one
whole-slice block item, or the chunk items of a giant slice; the chunks of a giant slice tile its level-1
node range without gap or overlap and there are ceil(nonzeros / chunk) of them; the light list is ordered
by falling size class; the light items tile the light list in groups of one slice per warp; the counts
agree with const_csf_bin_counts.  Slice sizes come from the COO input on the host, so nothing here is
derived from the arrays under test except the CSF positions they must agree with.
"""
import numpy as np
import pytest

import paper_2401_04836_b200 as cb
from workloads import make_config, ttmc3_workload, ttmc4_workload
from tests.gpu_util import build_csf

pytestmark = pytest.mark.gpu

WARPS_PER_LIGHT_ITEM = 2
SETTINGS = [None, (1 << 40, 1 << 41, 1 << 30), (1, 1 << 40, 1 << 30), (1, 2, 700), (300, 3000, 1500), (64, 64, 64)]
DEFAULTS = (4096, 16384, 8192)


def check_lists(h, op, mode_order, bins):
    light_max, heavy_max, chunk = bins
    root = op.coords[mode_order[0]]
    present = np.unique(root)                                   # slice s of the CSF holds coordinate present[s]
    size = np.bincount(root, minlength=op.dims[mode_order[0]])[present]
    n0 = present.size
    slice_ptr, light_list, items = (t.cpu().numpy() for t in cb.const_csf_work_lists(h))
    pos1 = cb.const_csf_level(h, 1)[0].cpu().numpy()
    counts = cb.const_csf_bin_counts(h)

    np.testing.assert_array_equal(np.diff(slice_ptr), size)     # leaf offsets of the slices
    assert slice_ptr[0] == 0 and slice_ptr[-1] == op.nnz

    want_light = np.nonzero(size <= light_max)[0]
    want_heavy = np.nonzero((size > light_max) & (size <= heavy_max))[0]
    want_giant = np.nonzero(size > heavy_max)[0]
    assert counts == {"light": want_light.size, "heavy": want_heavy.size, "giant": want_giant.size,
                      "items": items.shape[0]}

    # light list: every light slice once, larger size classes first
    np.testing.assert_array_equal(np.sort(light_list), want_light)
    cls = np.floor(np.log2(np.maximum(size[light_list], 1))).astype(int)
    assert np.all(np.diff(cls) <= 0)

    kind = items[:, 3]
    seen = np.zeros(n0, dtype=int)
    seen[light_list] += 1
    # block items: one per heavy slice, covering all of its level-1 nodes
    blk = items[kind == 1]
    np.testing.assert_array_equal(np.sort(blk[:, 0]), want_heavy)
    np.testing.assert_array_equal(blk[:, 1], pos1[blk[:, 0]])
    np.testing.assert_array_equal(blk[:, 2], pos1[blk[:, 0] + 1])
    seen[blk[:, 0]] += 1
    # chunk items: the chunks of a giant slice tile [pos1[s], pos1[s + 1]) in order
    chk = items[kind == 2]
    assert set(chk[:, 0].tolist()) == set(want_giant.tolist())
    for s in want_giant:
        mine = chk[chk[:, 0] == s]
        assert mine.shape[0] == -(-int(size[s]) // chunk)
        mine = mine[np.argsort(mine[:, 1], kind="stable")]
        assert mine[0, 1] == pos1[s] and mine[-1, 2] == pos1[s + 1]
        np.testing.assert_array_equal(mine[1:, 1], mine[:-1, 2])          # no gap, no overlap
        assert np.all(mine[:, 2] >= mine[:, 1])
        seen[s] += 1
    assert np.all(seen == 1)
    # light items: groups of consecutive light-list entries, one slice per warp
    lit = items[kind == 0]
    lit = lit[np.argsort(lit[:, 0])]
    assert lit.shape[0] == -(-want_light.size // WARPS_PER_LIGHT_ITEM)
    if lit.shape[0]:
        np.testing.assert_array_equal(lit[:, 0], np.arange(lit.shape[0]) * WARPS_PER_LIGHT_ITEM)
        assert np.all(lit[:-1, 1] == WARPS_PER_LIGHT_ITEM) and lit[:, 1].sum() == want_light.size
    assert items.shape[0] == blk.shape[0] + chk.shape[0] + lit.shape[0]


@pytest.mark.parametrize("bins", SETTINGS)
def test_work_lists_order3(bins):
    w = ttmc3_workload((500, 300, 700), 120_000, 16, slice_s=1.1, inner_s=0.9, value="unit", config_id=2)
    X = w.sparse["X"]
    h = build_csf(X, (0, 1, 2))
    if bins is not None:
        cb.const_csf_set_bins(h, *bins)
    check_lists(h, X, (0, 1, 2), bins or DEFAULTS)


def test_work_lists_after_rebinning_twice_and_other_root():
    w = ttmc3_workload((60, 500, 400), 90_000, 8, slice_s=1.3, inner_s=None, value="pm1", config_id=21)
    X = w.sparse["X"]
    h = build_csf(X, (1, 0, 2))                                 # mode 1 at the root
    for bins in [(100, 1000, 300), (1, 2, 50), (1 << 40, 1 << 41, 1 << 30), (20, 400, 400)]:
        cb.const_csf_set_bins(h, *bins)
        check_lists(h, X, (1, 0, 2), bins)


def test_work_lists_order4():
    w = ttmc4_workload((300, 40, 30, 50), 80_000, 8, slice_s=1.0, value="pm1", config_id=3)
    X = w.sparse["X"]
    h = build_csf(X, (0, 1, 2, 3))
    check_lists(h, X, (0, 1, 2, 3), DEFAULTS)
    cb.const_csf_set_bins(h, 50, 500, 200)
    check_lists(h, X, (0, 1, 2, 3), (50, 500, 200))


def test_work_lists_config2_quarter_scale_default_bins():
    w = make_config(2, scale=0.25)                              # 19 M nonzeros: the three bins are all populated
    X = w.sparse["X"]
    h = build_csf(X, (0, 1, 2))
    check_lists(h, X, (0, 1, 2), DEFAULTS)
