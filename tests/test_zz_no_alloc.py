"""const_csf_build_noalloc against the CSF oracle and against const_csf_build, and the property it exists for.

The no-allocation entry point is for callers that cannot obtain device memory when they need a CSF
tensor (a plug-in confined to a host application's arena, a latency-critical loop that must stay
clear of the driver's allocator, a process at its memory limit).  Its temporaries live in one static
device array shared by all calls, so the test makes calls in a row -- the second on a smaller,
different tensor, so that stale contents of the array would show -- and compares every array bit
for bit with the CPU oracle's CSF (oracle/csf.py) and with what const_csf_build produces for the same
input.  It also checks that a call after the first leaves the amount of free device memory, and the
counters of torch's caching allocator, exactly where they were.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from oracle import csf as ocsf
from workloads import generators as gen
from tests.gpu_util import build_csf, csf_to_host, to_dev

pytestmark = pytest.mark.gpu


def _noalloc(op, mode_order):
    order, nnz = len(op.dims), op.nnz
    coords = [to_dev(c.astype(np.int32)) for c in op.coords]
    vals = to_dev(op.vals)
    # the caller owns the outputs; poison them so that anything left unwritten shows up
    pos = [torch.full((2 if l == 0 else nnz + 1,), -7, dtype=torch.int32, device="cuda") for l in range(order)]
    crd = [torch.full((max(nnz, 1),), -7, dtype=torch.int32, device="cuda") for l in range(order)]
    vout = torch.full((max(nnz, 1),), float("nan"), dtype=vals.dtype, device="cuda")
    sizes = cb.const_csf_build_noalloc(coords, vals, op.dims, mode_order, pos, crd, vout)
    host_pos = [pos[l][: (2 if l == 0 else sizes[l - 1] + 1)].cpu().numpy() for l in range(order)]
    host_crd = [crd[l][: sizes[l]].cpu().numpy() for l in range(order)]
    return sizes, host_pos, host_crd, vout[:nnz].cpu().numpy()


def _same_as_handle_build(op, mode_order):
    sizes, pos, crd, vals = _noalloc(op, mode_order)
    for what, (ref_pos, ref_crd, ref_vals) in (("oracle", ocsf.build(op.coords, op.vals, mode_order)),
                                               ("const_csf_build", csf_to_host(build_csf(op, mode_order)))):
        assert sizes == [len(c) for c in ref_crd], what
        for l in range(len(mode_order)):
            np.testing.assert_array_equal(pos[l], ref_pos[l], err_msg=f"pos level {l} vs {what}")
            np.testing.assert_array_equal(crd[l], ref_crd[l], err_msg=f"crd level {l} vs {what}")
        assert vals.dtype == ref_vals.dtype and vals.tobytes() == ref_vals.tobytes(), what


def test_two_calls_in_a_row_match_const_csf_build():
    rng = np.random.default_rng(42)
    first = gen._uniform_tensor((300, 1000, 777), 200_003, rng, "pm1", np.float32)      # 49 tiles, ragged tail
    second = gen._uniform_tensor((64, 50, 40, 30), 9_001, rng, "normal", np.float64)    # smaller, other dtype and order
    _same_as_handle_build(first, (0, 1, 2))
    _same_as_handle_build(second, (2, 0, 3, 1))
    _same_as_handle_build(first, (2, 1, 0))                                             # and back to the large one


def test_a_call_after_the_first_obtains_no_device_memory():
    rng = np.random.default_rng(7)
    op = gen._uniform_tensor((200, 300, 150), 150_001, rng, "normal", np.float32)
    order, nnz = 3, op.nnz
    coords = [to_dev(c.astype(np.int32)) for c in op.coords]
    vals = to_dev(op.vals)
    pos = [torch.empty(2 if l == 0 else nnz + 1, dtype=torch.int32, device="cuda") for l in range(order)]
    crd = [torch.empty(nnz, dtype=torch.int32, device="cuda") for l in range(order)]
    vout = torch.empty_like(vals)
    # the first call on a device resolves the address of the static array (and, with lazy module loading,
    # is when the driver places the array and the kernels on the device)
    cb.const_csf_build_noalloc(coords, vals, op.dims, (0, 1, 2), pos, crd, vout)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    stats_before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(),
                    torch.cuda.memory_stats().get("num_alloc_retries", 0),
                    torch.cuda.memory_stats().get("allocation.all.allocated", 0))
    for mode_order in ((2, 0, 1), (1, 2, 0)):
        sizes = cb.const_csf_build_noalloc(coords, vals, op.dims, mode_order, pos, crd, vout)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        stats_after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(),
                       torch.cuda.memory_stats().get("num_alloc_retries", 0),
                       torch.cuda.memory_stats().get("allocation.all.allocated", 0))
        assert free_after == free_before, (free_before, free_after)
        assert stats_after == stats_before
    # and the result of that last call is right
    opos, ocrd, ovals = ocsf.build(op.coords, op.vals, (1, 2, 0))
    assert sizes == [len(c) for c in ocrd]
    for l in range(order):
        np.testing.assert_array_equal(crd[l][: sizes[l]].cpu().numpy(), ocrd[l])
        np.testing.assert_array_equal(pos[l][: (2 if l == 0 else sizes[l - 1] + 1)].cpu().numpy(), opos[l])
    assert vout.cpu().numpy().tobytes() == ovals.tobytes()


def test_limit_and_errors():
    rng = np.random.default_rng(1)
    too_big = gen._uniform_tensor((1000, 1000, 1000), 262_145, rng, "pm1", np.float32)
    with pytest.raises(cb.ConstError) as e:
        _noalloc(too_big, (0, 1, 2))
    assert e.value.status == 6                                                          # CONST_ERR_WORKSPACE
    S = gen.SparseOperand
    dup = S([np.array([1, 1], np.int32)] * 3, np.ones(2, np.float32), (4, 4, 4))
    with pytest.raises(cb.ConstError) as e:
        _noalloc(dup, (0, 1, 2))
    assert e.value.status == 4
    at_limit = gen._uniform_tensor((1000, 1000, 1000), 262_144, rng, "pm1", np.float32)
    _same_as_handle_build(at_limit, (1, 2, 0))
